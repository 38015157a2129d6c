// C ABI of the AdaSD hot path (see include/adasd.h): context management, argument
// validation and kernel launches.  No torch types, no CPU fallback: without a CUDA
// device every call fails with ADASD_ERR_CUDA.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "adasd_rows.cuh"
#include "adasd_cluster.cuh"
#include "adasd_spec.cuh"
#include "adasd_draft.cuh"
#include "adasd_vanilla.cuh"
#include "adasd_modes.cuh"

using namespace adasd;

struct adasd_ctx {
    adasd_config cfg;
    State st;
    Scratch sc;
    std::vector<void*> allocs;
    int sm_count;
    // warp-specialised verification kernel, one configuration per mode (AdaSD, vanilla);
    // iter == 0 means not usable for this V / dtype
    struct Fast {
        int iter;             // iterations per warp and row (template parameter)
        int cs;               // CTAs per cluster
        int smem;             // dynamic shared memory per CTA
        ClusterGeom geom;
    } fast[2];
    bool draft_stream;        // the streaming draft kernel is usable for this V / dtype
    bool lse_stream;          // ... and so is the row log-sum-exp kernel of the vanilla mode
    bool sample_stream;       // ... and its sampling kernel (the vocabulary fits its chunk tables)
    bool cut_hist;            // the one-pass cutoff kernel got its 128 KB of shared memory
    // adjusted distribution (adasd_set_warpers) and the per-row cutoffs a call works out
    float temperature;
    int32_t top_k;
    float top_p;
    float* cut_t;             // [B,Kmax+1]
    float* cut_d;             // [B,Kmax]
    float* cut_row;           // [B] draft step
    bool cuts_on() const { return (top_k > 0 && top_k < cfg.V) || top_p < 1.f; }
    bool warp_on() const { return cuts_on() || temperature != 1.f; }
};

namespace {

#define CUDA_TRY(expr)                         \
    do {                                       \
        cudaError_t e__ = (expr);              \
        if (e__ != cudaSuccess) return ADASD_ERR_CUDA; \
    } while (0)

template <typename T>
int dev_alloc(adasd_ctx* c, T** p, size_t n) {
    void* q = nullptr;
    if (cudaMalloc(&q, n * sizeof(T)) != cudaSuccess) return ADASD_ERR_CUDA;
    if (cudaMemset(q, 0, n * sizeof(T)) != cudaSuccess) return ADASD_ERR_CUDA;
    c->allocs.push_back(q);
    *p = static_cast<T*>(q);
    return ADASD_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t elt_size(int dtype) { return dtype == ADASD_BF16 ? 2 : 4; }

// NULL counts as aligned: whether a pointer may be NULL is checked where it is used.
inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline bool aligned4(std::initializer_list<const void*> ps) {
    for (const void* p : ps)
        if (!aligned_to(p, 4)) return false;
    return true;
}

// The hot calls launch on the calling thread's current device with this context's pointers:
// refuse when that is another GPU.
int check_device(const adasd_ctx* c) {
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) {
        cudaGetLastError();
        return ADASD_ERR_CUDA;
    }
    return cur == c->cfg.device ? ADASD_OK : ADASD_ERR_DEVICE;
}

// Rows can take 16-byte loads when the base and every stride are 16-byte multiples.
inline bool vec_ok(const void* base, int dtype, std::initializer_list<long long> strides) {
    if (!aligned16(base)) return false;
    for (long long s : strides)
        if ((s * (long long)elt_size(dtype)) % 16 != 0) return false;
    return true;
}

int pick_cluster(const adasd_ctx* c, long long rows) {
    if (c->cfg.cluster_size > 0) return c->cfg.cluster_size;
    const long long want = 2LL * c->sm_count;
    for (int cs = 1; cs <= kMaxCluster; cs *= 2)
        if (rows * cs >= want) return cs;
    return kMaxCluster;
}

template <typename P>
int launch_cluster(void (*kernel)(P), const P& params, long long clusters, int cs,
                   cudaStream_t stream) {
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3((unsigned)(clusters * cs), 1, 1);
    lc.blockDim = dim3(kThreads, 1, 1);
    lc.dynamicSmemBytes = 0;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    CUDA_TRY(cudaLaunchKernelEx(&lc, kernel, params));
    return ADASD_OK;
}

// ---- warp-specialised verification kernel: configuration and launch ----------------------
template <typename K>
int kernel_occupancy(K kern, int threads, int cs, int smem) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3((unsigned)(cs * 64), 1, 1);
    lc.blockDim = dim3((unsigned)threads, 1, 1);
    lc.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &lc) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

template <typename K>
int kernel_static_smem(K kern) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return (int)fa.sharedSizeBytes;
}

// Both modes run the warp-specialised kernel.
template <int ITER, int MODE>
int fast_occupancy(int cs, int smem) {
    return kernel_occupancy(spec_verify_kernel<ITER, MODE>, kSThreads, cs, smem);
}
template <int ITER, int MODE>
int fast_static_smem() {
    return kernel_static_smem(spec_verify_kernel<ITER, MODE>);
}

#define ADASD_ITER_SWITCH(iter, CALL, fail)  \
    switch (iter) {                          \
        case 1: return CALL(1);              \
        case 2: return CALL(2);              \
        case 3: return CALL(3);              \
        case 4: return CALL(4);              \
        case 5: return CALL(5);              \
        case 6: return CALL(6);              \
        case 7: return CALL(7);              \
        case 8: return CALL(8);              \
        case 9: return CALL(9);              \
        case 10: return CALL(10);            \
        default: return fail;                \
    }

template <int MODE>
int fast_occupancy_iter(int iter, int cs, int smem) {
#define CALL(I) fast_occupancy<I, MODE>(cs, smem)
    ADASD_ITER_SWITCH(iter, CALL, 0)
#undef CALL
}
template <int MODE>
int fast_static_smem_iter(int iter) {
#define CALL(I) fast_static_smem<I, MODE>()
    ADASD_ITER_SWITCH(iter, CALL, -1)
#undef CALL
}

// Chooses, for one mode, the cluster size that covers the most SMs among those whose per-CTA
// slice fits on chip: two position buffers per compute warp, iter * 512 bytes per row (the
// 2^t values live in registers or are worked out again).  bf16 rows of a multiple of 8
// elements only.
template <int MODE>
void fast_setup_mode(adasd_ctx* c, size_t smem_optin) {
    adasd_ctx::Fast& f = c->fast[MODE];
    f.iter = 0;
    const int V = c->cfg.V;
    if (c->cfg.dtype != ADASD_BF16 || (V & 7) != 0 || V < 8192) return;
    const int NU = V >> 3;
    int best_score = 0;
    for (int cs = kCMaxCluster; cs >= 1; --cs) {
        if (c->cfg.cluster_size != 0 && c->cfg.cluster_size != cs) continue;
        const int ncu = (NU + cs - 1) / cs, nwi = (ncu + 31) / 32;
        const int I_lo = nwi / kSW, rem = nwi % kSW, iter = I_lo + (rem ? 1 : 0);
        if (iter < 1 || iter > kSMaxIter) continue;
        const int st = fast_static_smem_iter<MODE>(iter);
        if (st < 0) continue;
        const int smem = nwi * 2048;      // two position buffers: 512 bytes per row and warp-iteration
        if (smem > (int)smem_optin - st - 1024) continue;
        const int ncl = fast_occupancy_iter<MODE>(iter, cs, smem);
        const int score = ncl * cs;
        if (score > best_score) {
            best_score = score;
            f.iter = iter;
            f.cs = cs;
            f.smem = smem;
            f.geom.ncl = ncl;
        }
    }
}
void fast_setup(adasd_ctx* c, size_t smem_optin) {
    fast_setup_mode<MODE_ADASD>(c, smem_optin);
    fast_setup_mode<MODE_VANILLA>(c, smem_optin);
    // streaming draft kernel: bf16 rows of a multiple of 8 logits, two 4 KB buffers per warp
    c->draft_stream = false;
    c->lse_stream = false;
    c->sample_stream = false;
    c->cut_hist = cudaFuncSetAttribute(row_cutoff_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kHistWords * 4) == cudaSuccess;
    if (!c->cut_hist) cudaGetLastError();
    const int V = c->cfg.V;
    if (c->cfg.dtype == ADASD_BF16 && (V & 7) == 0 && V >= 8192 &&
        (V >> 3) <= kDMaxP * kDW * kDMaxChunks * kDChunkUnits) {
        if (cudaFuncSetAttribute(draft_stream_kernel<kDW, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDW * 2 * kDChunkBytes) == cudaSuccess &&
            cudaFuncSetAttribute(draft_stream_kernel<kDWBig, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDWBig * 2 * kDChunkBytes) == cudaSuccess &&
            cudaFuncSetAttribute(draft_stream_kernel<kDW, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDW * 2 * kDChunkBytes) == cudaSuccess &&
            cudaFuncSetAttribute(draft_stream_kernel<kDWBig, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDWBig * 2 * kDChunkBytes) == cudaSuccess)
            c->draft_stream = true;
        else
            cudaGetLastError();
        if (cudaFuncSetAttribute(row_lse_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kLW * 2 * kLChunkBytes) == cudaSuccess &&
            cudaFuncSetAttribute(row_lse_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kLW * 2 * kLChunkBytes) == cudaSuccess)
            c->lse_stream = true;
        else
            cudaGetLastError();
        if (V <= kVMaxV) {
            if (cudaFuncSetAttribute(vanilla_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kVW * 4 * kVChunkBytes) == cudaSuccess)
                c->sample_stream = true;
            else
                cudaGetLastError();
        }
    }
}

// CTAs per row for the streaming draft kernel: enough to fill the SMs, and few enough chunks
// per warp for its tables
int draft_stream_p(const adasd_ctx* c) {
    const int NU = c->cfg.V >> 3;
    int P = 1;
    if (c->cfg.cluster_size == 1 || c->cfg.cluster_size == 2 || c->cfg.cluster_size == 4 ||
        c->cfg.cluster_size == 8)
        P = c->cfg.cluster_size;
    else
        while (P < kDMaxP && (long long)c->cfg.B * P * 4 < 3LL * c->sm_count) P *= 2;
    while (P < kDMaxP && (NU + P * kDW - 1) / (P * kDW) > kDMaxChunks * kDChunkUnits) P *= 2;
    return P;
}

template <int ITER, int MODE, bool WARPED>
int fast_launch(adasd_ctx* c, const VerifyParams& p, cudaStream_t stream) {
    const long long positions = (long long)p.B * (p.Kmax + 1);
    const adasd_ctx::Fast& f = c->fast[MODE];
    ClusterGeom gq = f.geom;
    if (positions < gq.ncl) gq.ncl = (int)positions;
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3((unsigned)(gq.ncl * f.cs), 1, 1);
    lc.blockDim = dim3((unsigned)kSThreads, 1, 1);
    lc.dynamicSmemBytes = (size_t)f.smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)f.cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (WARPED) {
        // the instantiation for adjusted distributions: same footprint, its own attribute
        CUDA_TRY(cudaFuncSetAttribute(spec_verify_kernel<ITER, MODE, WARPED>, cudaFuncAttributeMaxDynamicSharedMemorySize, f.smem));
    }
    CUDA_TRY(cudaLaunchKernelEx(&lc, spec_verify_kernel<ITER, MODE, WARPED>, p, gq));
    return ADASD_OK;
}

template <int MODE>
int fast_launch_iter(adasd_ctx* c, const VerifyParams& p, cudaStream_t stream) {
    if (c->warp_on()) {
#define CALL(I) fast_launch<I, MODE, true>(c, p, stream)
        ADASD_ITER_SWITCH(c->fast[MODE].iter, CALL, ADASD_ERR_SHAPE)
#undef CALL
    }
#define CALL(I) fast_launch<I, MODE, false>(c, p, stream)
    ADASD_ITER_SWITCH(c->fast[MODE].iter, CALL, ADASD_ERR_SHAPE)
#undef CALL
}

int check_strides(const adasd_ctx* c, long long seq, long long row) {
    if (row < c->cfg.V || seq < 0) return ADASD_ERR_SHAPE;
    return ADASD_OK;
}

int fill_verify_params(adasd_ctx* ctx, VerifyParams& p, const void* zd, const void* zt,
                       int64_t d_seq, int64_t d_row, int64_t t_seq, int64_t t_row,
                       const int32_t* x, const int32_t* draft_len) {
    if (!ctx || !zd || !zt || !x) return ADASD_ERR_NULL;
    int rc;
    if ((rc = check_device(ctx)) != ADASD_OK) return rc;
    const size_t es = elt_size(ctx->cfg.dtype);
    if (!aligned_to(zd, es) || !aligned_to(zt, es) || !aligned4({x, draft_len})) return ADASD_ERR_ALIGN;
    if ((rc = check_strides(ctx, d_seq, d_row)) != ADASD_OK) return rc;
    if ((rc = check_strides(ctx, t_seq, t_row)) != ADASD_OK) return rc;
    memset(&p, 0, sizeof(p));
    p.zd = zd;
    p.zt = zt;
    p.d_seq = d_seq;
    p.d_row = d_row;
    p.t_seq = t_seq;
    p.t_row = t_row;
    p.x = x;
    p.draft_len = draft_len;
    p.sc = ctx->sc;
    p.st = ctx->st;
    p.B = ctx->cfg.B;
    p.V = ctx->cfg.V;
    p.Kmax = ctx->cfg.Kmax;
    p.tail.Kmax = ctx->cfg.Kmax;
    p.tail.min_samples = ctx->cfg.min_kde_samples;
    p.tail.bw_rule = ctx->cfg.kde_bandwidth;
    p.tail.reject_rule = ctx->cfg.reject_rule;
    p.tail.update = 0;
    p.inv_temp = 1.f / ctx->temperature;
    p.c1 = kLog2e / ctx->temperature;
    if (ctx->cuts_on()) {
        p.cut_t = ctx->cut_t;
        p.cut_d = ctx->cut_d;
    }
    return ADASD_OK;
}

// One cutoff logit per needed row (top-k / top-p of the adjusted distribution).
int launch_cutoffs(adasd_ctx* ctx, const void* z, long long seq_stride, long long row_stride, int R, int extra,
                   const int32_t* draft_len, const uint8_t* active, float* cut, cudaStream_t stream) {
    CutParams c;
    memset(&c, 0, sizeof(c));
    c.z = z;
    c.seq_stride = seq_stride;
    c.row_stride = row_stride;
    c.draft_len = draft_len;
    c.active = active;
    c.cut = cut;
    c.status = ctx->st.status;
    c.B = ctx->cfg.B;
    c.R = R;
    c.V = ctx->cfg.V;
    c.extra = extra;
    c.c1 = 1.4426950408889634 / (double)ctx->temperature;
    c.top_k = ctx->top_k;
    c.top_p = ctx->top_p;
    const long long rows = (long long)c.B * R;
    const bool vec = vec_ok(z, ctx->cfg.dtype, {seq_stride, row_stride});
    if (ctx->cfg.dtype == ADASD_BF16 && vec && ctx->cut_hist) {
        // one pass per row over a histogram of the 65536 bf16 values; a row it cannot do (a value
        // that occurs 65536 times or more) is left flagged for the radix kernel
        const int g1 = (int)std::min<long long>(rows, (long long)ctx->sm_count);
        row_cutoff_hist_kernel<<<g1, kHistThreads, kHistWords * 4, stream>>>(c);
        CUDA_TRY(cudaGetLastError());
        c.only_flagged = 1;
    }
    const int grid = (int)std::min<long long>(rows, 2LL * ctx->sm_count);
    if (ctx->cfg.dtype == ADASD_BF16) {
        if (vec) row_cutoff_kernel<__nv_bfloat16, true><<<grid, kCutThreads, 0, stream>>>(c);
        else row_cutoff_kernel<__nv_bfloat16, false><<<grid, kCutThreads, 0, stream>>>(c);
    } else {
        if (vec) row_cutoff_kernel<float, true><<<grid, kCutThreads, 0, stream>>>(c);
        else row_cutoff_kernel<float, false><<<grid, kCutThreads, 0, stream>>>(c);
    }
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

template <int MODE>
int launch_verify(adasd_ctx* ctx, const VerifyParams& p, cudaStream_t stream) {
    const long long positions = (long long)p.B * (p.Kmax + 1);
    const int cs = pick_cluster(ctx, positions);
    const bool vec = vec_ok(p.zd, ctx->cfg.dtype, {p.d_seq, p.d_row}) &&
                     vec_ok(p.zt, ctx->cfg.dtype, {p.t_seq, p.t_row});
    if (ctx->cuts_on()) {
        if (int rc = launch_cutoffs(ctx, p.zt, p.t_seq, p.t_row, p.Kmax + 1, 1, p.draft_len, nullptr, ctx->cut_t, stream))
            return rc;
        if (int rc = launch_cutoffs(ctx, p.zd, p.d_seq, p.d_row, p.Kmax, 0, p.draft_len, nullptr, ctx->cut_d, stream))
            return rc;
    }
    if (vec && ctx->fast[MODE].iter > 0) {
        // Vanilla mode with enough rows to fill the GPU: log-sum-exps of all rows in one light
        // streaming pass, the accept test per sequence, then the sampling of one position per
        // sequence.  With fewer rows than CTA slots of the streaming pass: everything in the one
        // cluster kernel.
        const long long rows = (long long)p.B * (2 * p.Kmax + 1);
        if (MODE == MODE_VANILLA && ctx->lse_stream && ctx->sample_stream && rows >= 2LL * ctx->sm_count) {
            LseParams lp;
            memset(&lp, 0, sizeof(lp));
            lp.zd = p.zd;
            lp.zt = p.zt;
            lp.d_seq = p.d_seq;
            lp.d_row = p.d_row;
            lp.t_seq = p.t_seq;
            lp.t_row = p.t_row;
            lp.draft_len = p.draft_len;
            lp.lse_d = p.sc.lse_d;
            lp.lse_t = p.sc.lse_t;
            lp.status = p.st.status;
            lp.B = p.B;
            lp.V = p.V;
            lp.Kmax = p.Kmax;
            lp.c1 = p.c1;
            lp.cut_t = p.cut_t;
            lp.cut_d = p.cut_d;
            if (ctx->warp_on()) row_lse_kernel<true><<<2 * ctx->sm_count, kLW * 32, kLW * 2 * kLChunkBytes, stream>>>(lp);
            else row_lse_kernel<false><<<2 * ctx->sm_count, kLW * 32, kLW * 2 * kLChunkBytes, stream>>>(lp);
            CUDA_TRY(cudaGetLastError());
            vanilla_accept_kernel<<<(p.B + 3) / 4, 128, 0, stream>>>(p, p.sc.only_pos);     // one warp per sequence
            CUDA_TRY(cudaGetLastError());
            // one CTA per sequence streams the row pair of its one position
            vanilla_sample_kernel<<<p.B, kVW * 32, kVW * 4 * kVChunkBytes, stream>>>(p, p.sc.only_pos);
            CUDA_TRY(cudaGetLastError());
            return ADASD_OK;
        }
        return fast_launch_iter<MODE>(ctx, p, stream);
    }
    if (ctx->cfg.dtype == ADASD_BF16) {
        return vec ? launch_cluster(verify_kernel<__nv_bfloat16, true, MODE>, p, positions, cs, stream)
                   : launch_cluster(verify_kernel<__nv_bfloat16, false, MODE>, p, positions, cs, stream);
    }
    return vec ? launch_cluster(verify_kernel<float, true, MODE>, p, positions, cs, stream)
               : launch_cluster(verify_kernel<float, false, MODE>, p, positions, cs, stream);
}

// The most probable token of every needed row (greedy drafting and greedy verification).
int launch_argmax(adasd_ctx* ctx, const ArgmaxParams& a, cudaStream_t stream) {
    const long long rows = (long long)a.B * a.R;
    const unsigned grid = (unsigned)std::min<long long>(rows, 4LL * ctx->sm_count);
    const bool vec = vec_ok(a.z, ctx->cfg.dtype, {a.seq_stride, a.row_stride});
    if (ctx->cfg.dtype == ADASD_BF16) {
        if (vec) row_argmax_kernel<__nv_bfloat16, true><<<grid, kAThreads, 0, stream>>>(a);
        else row_argmax_kernel<__nv_bfloat16, false><<<grid, kAThreads, 0, stream>>>(a);
    } else {
        if (vec) row_argmax_kernel<float, true><<<grid, kAThreads, 0, stream>>>(a);
        else row_argmax_kernel<float, false><<<grid, kAThreads, 0, stream>>>(a);
    }
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (ok && prev >= 0) {
            int cur = -1;
            if (cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
        }
    }
};

constexpr size_t kExportHeader = 24;

}  // namespace

// ---- allocation-free vanilla verification -------------------------------------------
// Scratch of adasd_vanilla_verify_static: lives in the library image, one copy per GPU
// that loads it, shared by every call.  Words: per-candidate accept flags, per-position
// candidate tokens, per-sequence arrival counters, one status word.
static __device__ __align__(256) uint32_t g_static_scratch[2 * ADASD_STATIC_MAX_POSITIONS +
                                                           ADASD_STATIC_MAX_B + 64];

namespace {
constexpr int kMaxDevices = 64;
struct StaticSetup {
    uint32_t* base = nullptr;   // device address of g_static_scratch on this device
    int sm_count = 0;
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;

// Device address of the scratch array on the CURRENT device.  The array's name is only a
// host-side handle: the address a kernel can use comes from cudaGetSymbolAddress, asked
// once per device with that device current.
int static_setup(int dev, StaticSetup& out) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup& s = g_static_setup[dev];
    if (!s.base) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return ADASD_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return ADASD_ERR_CUDA;
        }
        s.sm_count = sms;
        s.base = static_cast<uint32_t*>(ptr);
    }
    out = s;
    return ADASD_OK;
}
}  // namespace

extern "C" {

int adasd_create(adasd_ctx** out, const adasd_config* cfg) {
    if (!out || !cfg) return ADASD_ERR_NULL;
    *out = nullptr;
    if (cfg->B < 1 || cfg->V < 1 || cfg->Kmax < 1 || cfg->Kmax > ADASD_KMAX_LIMIT ||
        cfg->list_capacity < 1)
        return ADASD_ERR_SHAPE;
    if ((long long)cfg->B * (cfg->Kmax + 1) > 0x3FFFFFFFLL) return ADASD_ERR_SHAPE;
    if (cfg->dtype != ADASD_BF16 && cfg->dtype != ADASD_FP32) return ADASD_ERR_DTYPE;
    if (cfg->kde_bandwidth < 0 || cfg->kde_bandwidth > 1 || cfg->reject_rule < 0 ||
        cfg->reject_rule > 1)
        return ADASD_ERR_DTYPE;
    if (cfg->cluster_size < 0 || cfg->cluster_size > kMaxCluster) return ADASD_ERR_SHAPE;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev)
        return ADASD_ERR_CUDA;
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return ADASD_ERR_CUDA;

    adasd_ctx* c = new (std::nothrow) adasd_ctx();
    if (!c) return ADASD_ERR_CUDA;
    c->cfg = *cfg;
    if (c->cfg.min_kde_samples < 2) c->cfg.min_kde_samples = 2;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) {
        delete c;
        return ADASD_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    memset(&c->st, 0, sizeof(c->st));
    memset(&c->sc, 0, sizeof(c->sc));

    const size_t B = (size_t)cfg->B, K = (size_t)cfg->Kmax, cap = (size_t)cfg->list_capacity;
    int rc = ADASD_OK;
    State& s = c->st;
    Scratch& t = c->sc;
    s.cap = cfg->list_capacity;
#define ALLOC(ptr, n)                                        \
    if (rc == ADASD_OK) rc = dev_alloc(c, &(ptr), (size_t)(n))
    ALLOC(s.T_G, B);
    ALLOC(s.sumE, B);
    ALLOC(s.nE, B);
    ALLOC(s.nA, B);
    ALLOC(s.nR, B);
    ALLOC(s.sumA, B);
    ALLOC(s.sumA2, B);
    ALLOC(s.sumR, B);
    ALLOC(s.sumR2, B);
    ALLOC(s.LE, B * cap);
    ALLOC(s.LA, B * cap);
    ALLOC(s.LR, B * cap);
    ALLOC(s.status, 1);
    ALLOC(t.H_d, B * K);
    ALLOC(t.H_t, B * (K + 1));
    ALLOC(t.lse_d, B * K);
    ALLOC(t.lse_t, B * (K + 1));
    ALLOC(t.jsd, B * K);
    ALLOC(t.dist, B * K);
    ALLOC(t.p_acc, B * K);
    ALLOC(t.y, B * (K + 1));
    ALLOC(t.van_flag, B * K);
    ALLOC(t.van_tok, B * (K + 1));
    ALLOC(t.ticket, B);
    ALLOC(t.only_pos, B);
    ALLOC(t.q_items, B);
    ALLOC(t.q_ctl, 4);
    ALLOC(c->cut_t, B * (K + 1));
    ALLOC(c->cut_d, B * K);
    ALLOC(c->cut_row, B);
#undef ALLOC
    c->temperature = 1.f;
    c->top_k = 0;
    c->top_p = 1.f;
    if (rc == ADASD_OK && cudaMemset(t.q_items, 0xFF, B * sizeof(int32_t)) != cudaSuccess) rc = ADASD_ERR_CUDA;
    if (rc == ADASD_OK) fast_setup(c, prop.sharedMemPerBlockOptin);
    if (rc == ADASD_OK && cudaDeviceSynchronize() != cudaSuccess) rc = ADASD_ERR_CUDA;
    if (rc != ADASD_OK) {
        for (void* q : c->allocs) cudaFree(q);
        delete c;
        return rc;
    }
    *out = c;
    return ADASD_OK;
}

int adasd_destroy(adasd_ctx* ctx) {
    if (!ctx) return ADASD_ERR_NULL;
    DeviceGuard guard(ctx->cfg.device);
    int rc = ADASD_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) rc = ADASD_ERR_CUDA;
    for (void* q : ctx->allocs)
        if (cudaFree(q) != cudaSuccess) rc = ADASD_ERR_CUDA;
    delete ctx;
    return rc;
}

int adasd_reset(adasd_ctx* ctx, const int32_t* seq_ids_dev, int32_t n, void* stream) {
    if (!ctx) return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned4({seq_ids_dev})) return ADASD_ERR_ALIGN;
    if (!seq_ids_dev) n = ctx->cfg.B;
    if (n < 0) return ADASD_ERR_SHAPE;
    if (n == 0) return ADASD_OK;
    reset_kernel<<<(n + 127) / 128, 128, 0, (cudaStream_t)stream>>>(ctx->st, seq_ids_dev, n,
                                                                    ctx->cfg.B);
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

// adasd_draft_entropy, optionally (expire_row >= 0) as the self-test of the bounded waits
static int draft_entropy_impl(adasd_ctx* ctx, const void* logits_dev, int64_t row_stride,
                              const float* u_dev, uint8_t* active_inout_dev, float* H_out_dev,
                              float* lse_out_dev, int32_t* token_out_dev, uint8_t* stop_out_dev,
                              int32_t* draft_len_inout_dev, void* stream, int32_t expire_row) {
    if (!ctx || !logits_dev || !H_out_dev) return ADASD_ERR_NULL;
    if (u_dev != nullptr && token_out_dev == nullptr) return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned_to(logits_dev, elt_size(ctx->cfg.dtype)) ||
        !aligned4({u_dev, H_out_dev, lse_out_dev, token_out_dev, draft_len_inout_dev}))
        return ADASD_ERR_ALIGN;
    if (row_stride < ctx->cfg.V) return ADASD_ERR_SHAPE;
    DraftParams p;
    memset(&p, 0, sizeof(p));
    p.z = logits_dev;
    p.row_stride = row_stride;
    p.u = u_dev;
    p.active = active_inout_dev;
    p.H_out = H_out_dev;
    p.lse_out = lse_out_dev;
    p.token_out = u_dev ? token_out_dev : nullptr;
    p.stop_out = stop_out_dev;
    p.draft_len = draft_len_inout_dev;
    p.st = ctx->st;
    p.B = ctx->cfg.B;
    p.V = ctx->cfg.V;
    p.expire_row = expire_row;
    p.inv_temp = 1.f / ctx->temperature;
    p.c1 = kLog2e / ctx->temperature;
    if (ctx->cuts_on()) p.cut = ctx->cut_row;
    const int cs = pick_cluster(ctx, p.B);
    const bool vec = vec_ok(logits_dev, ctx->cfg.dtype, {row_stride});
    if (expire_row >= 0 && !(vec && ctx->draft_stream && expire_row < ctx->cfg.B))
        return ADASD_ERR_SHAPE;                  // the self-test needs the streaming kernel
    cudaStream_t st = (cudaStream_t)stream;
    if (!u_dev && token_out_dev) {
        // greedy drafting: the most probable token of every active row, before the step below can
        // clear a row's entry in the active mask (the token that trips the stop check stays)
        ArgmaxParams a;
        memset(&a, 0, sizeof(a));
        a.z = logits_dev;
        a.seq_stride = row_stride;
        a.row_stride = 0;
        a.active = active_inout_dev;
        a.out = token_out_dev;
        a.status = ctx->st.status;
        a.B = ctx->cfg.B;
        a.R = 1;
        a.V = ctx->cfg.V;
        if (int rc = launch_argmax(ctx, a, st)) return rc;
    }
    if (ctx->cuts_on()) {
        if (int rc = launch_cutoffs(ctx, logits_dev, row_stride, 0, 1, 1, nullptr, active_inout_dev, ctx->cut_row, st))
            return rc;
    }
    if (vec && ctx->draft_stream) {
        const int P = draft_stream_p(ctx);
        // a grid of at most one CTA per SM runs 16 warps per CTA, a larger one 8 (two CTAs per SM)
        const bool big = (long long)p.B * P <= ctx->sm_count && P * kDWBig <= kDMaxEntries;
        const int W = big ? kDWBig : kDW;
        cudaLaunchConfig_t lc;
        memset(&lc, 0, sizeof(lc));
        lc.gridDim = dim3((unsigned)(p.B * P), 1, 1);
        lc.blockDim = dim3((unsigned)(W * 32), 1, 1);
        lc.dynamicSmemBytes = (size_t)(W * 2 * kDChunkBytes);
        lc.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)P;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // the launch may overlap the tail of the kernel ahead of it (the kernel waits before it
        // reads anything): draft steps come in runs of short calls
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = attr;
        lc.numAttrs = 2;
        const bool warped = ctx->warp_on();
        if (big) {
            if (warped) CUDA_TRY(cudaLaunchKernelEx(&lc, draft_stream_kernel<kDWBig, true>, p));
            else CUDA_TRY(cudaLaunchKernelEx(&lc, draft_stream_kernel<kDWBig, false>, p));
        } else {
            if (warped) CUDA_TRY(cudaLaunchKernelEx(&lc, draft_stream_kernel<kDW, true>, p));
            else CUDA_TRY(cudaLaunchKernelEx(&lc, draft_stream_kernel<kDW, false>, p));
        }
        return ADASD_OK;
    }
    if (ctx->cfg.dtype == ADASD_BF16)
        return vec ? launch_cluster(draft_kernel<__nv_bfloat16, true>, p, p.B, cs, st)
                   : launch_cluster(draft_kernel<__nv_bfloat16, false>, p, p.B, cs, st);
    return vec ? launch_cluster(draft_kernel<float, true>, p, p.B, cs, st)
               : launch_cluster(draft_kernel<float, false>, p, p.B, cs, st);
}

int adasd_draft_entropy(adasd_ctx* ctx, const void* logits_dev, int64_t row_stride,
                        const float* u_dev, uint8_t* active_inout_dev, float* H_out_dev,
                        float* lse_out_dev, int32_t* token_out_dev, uint8_t* stop_out_dev,
                        int32_t* draft_len_inout_dev, void* stream) {
    return draft_entropy_impl(ctx, logits_dev, row_stride, u_dev, active_inout_dev, H_out_dev, lse_out_dev,
                              token_out_dev, stop_out_dev, draft_len_inout_dev, stream, -1);
}

int adasd_selftest_expired_wait(adasd_ctx* ctx, const void* logits_dev, int64_t row_stride, int32_t row,
                                const float* u_dev, float* H_out_dev, int32_t* token_out_dev, void* stream) {
    if (row < 0) return ADASD_ERR_SHAPE;
    return draft_entropy_impl(ctx, logits_dev, row_stride, u_dev, nullptr, H_out_dev, nullptr, token_out_dev,
                              nullptr, nullptr, stream, row);
}

int adasd_verify(adasd_ctx* ctx, const void* draft_logits_dev, const void* target_logits_dev,
                 int64_t d_seq_stride, int64_t d_row_stride, int64_t t_seq_stride,
                 int64_t t_row_stride, const int32_t* draft_tokens_dev,
                 const int32_t* draft_len_dev, const float* u_target_dev,
                 const float* u_accept_dev, int32_t* accept_len_dev, int32_t* next_token_dev,
                 const adasd_round_record* record, uint32_t flags, void* stream) {
    VerifyParams p;
    int rc = fill_verify_params(ctx, p, draft_logits_dev, target_logits_dev, d_seq_stride,
                                d_row_stride, t_seq_stride, t_row_stride, draft_tokens_dev,
                                draft_len_dev);
    if (rc != ADASD_OK) return rc;
    if (!u_target_dev || !u_accept_dev || !accept_len_dev || !next_token_dev)
        return ADASD_ERR_NULL;
    if (!aligned4({u_target_dev, u_accept_dev, accept_len_dev, next_token_dev})) return ADASD_ERR_ALIGN;
    if (record && !aligned4({record->H_d, record->H_t, record->lse_d, record->lse_t, record->jsd,
                             record->dist, record->p_acc, record->y, record->draft_len,
                             record->accept_len, record->rejected}))
        return ADASD_ERR_ALIGN;
    if (flags & ~ADASD_FUSE_UPDATE) return ADASD_ERR_SHAPE;
    p.u_target = u_target_dev;
    p.u_accept = u_accept_dev;
    p.accept_len = accept_len_dev;
    p.next_token = next_token_dev;
    if (record) p.user = *record;
    p.tail.update = (flags & ADASD_FUSE_UPDATE) ? 1u : 0u;
    return launch_verify<MODE_ADASD>(ctx, p, (cudaStream_t)stream);
}

int adasd_update_thresholds(adasd_ctx* ctx, const adasd_round_record* record, void* stream) {
    if (!ctx || !record) return ADASD_ERR_NULL;
    if (!record->H_d || !record->dist || !record->draft_len || !record->accept_len ||
        !record->rejected)
        return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned4({record->H_d, record->dist, record->draft_len, record->accept_len, record->rejected}))
        return ADASD_ERR_ALIGN;
    const int B = ctx->cfg.B;
    update_kernel<<<(B + 127) / 128, 128, 0, (cudaStream_t)stream>>>(ctx->st, *record, B,
                                                                     ctx->cfg.Kmax);
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

int adasd_vanilla_verify(adasd_ctx* ctx, const void* draft_logits_dev,
                         const void* target_logits_dev, int64_t d_seq_stride,
                         int64_t d_row_stride, int64_t t_seq_stride, int64_t t_row_stride,
                         const int32_t* draft_tokens_dev, const int32_t* draft_len_dev,
                         const float* u_accept_dev, const float* u_resample_dev,
                         int32_t* accept_len_dev, int32_t* next_token_dev, float* alpha_out_dev,
                         void* stream) {
    VerifyParams p;
    int rc = fill_verify_params(ctx, p, draft_logits_dev, target_logits_dev, d_seq_stride,
                                d_row_stride, t_seq_stride, t_row_stride, draft_tokens_dev,
                                draft_len_dev);
    if (rc != ADASD_OK) return rc;
    if (!u_accept_dev || !u_resample_dev || !accept_len_dev || !next_token_dev)
        return ADASD_ERR_NULL;
    if (!aligned4({u_accept_dev, u_resample_dev, accept_len_dev, next_token_dev, alpha_out_dev}))
        return ADASD_ERR_ALIGN;
    p.u_accept = u_accept_dev;
    p.u_resample = u_resample_dev;
    p.accept_len = accept_len_dev;
    p.next_token = next_token_dev;
    p.alpha_out = alpha_out_dev;
    return launch_verify<MODE_VANILLA>(ctx, p, (cudaStream_t)stream);
}

int adasd_greedy_verify(adasd_ctx* ctx, const void* target_logits_dev, int64_t t_seq_stride,
                        int64_t t_row_stride, const int32_t* draft_tokens_dev,
                        const int32_t* draft_len_dev, int32_t* accept_len_dev, int32_t* next_token_dev,
                        int32_t* argmax_out_dev, void* stream) {
    if (!ctx || !target_logits_dev || !draft_tokens_dev || !accept_len_dev || !next_token_dev)
        return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned_to(target_logits_dev, elt_size(ctx->cfg.dtype)) ||
        !aligned4({draft_tokens_dev, draft_len_dev, accept_len_dev, next_token_dev, argmax_out_dev}))
        return ADASD_ERR_ALIGN;
    if (int rc = check_strides(ctx, t_seq_stride, t_row_stride)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const int B = ctx->cfg.B, K = ctx->cfg.Kmax;
    ArgmaxParams a;
    memset(&a, 0, sizeof(a));
    a.z = target_logits_dev;
    a.seq_stride = t_seq_stride;
    a.row_stride = t_row_stride;
    a.draft_len = draft_len_dev;
    a.out = ctx->sc.van_tok;                 // [B, Kmax + 1] scratch of the comparison modes
    a.status = ctx->st.status;
    a.B = B;
    a.R = K + 1;
    a.V = ctx->cfg.V;
    if (int rc = launch_argmax(ctx, a, st)) return rc;
    greedy_accept_kernel<<<(B + 127) / 128, 128, 0, st>>>(draft_tokens_dev, ctx->sc.van_tok, draft_len_dev,
                                                        accept_len_dev, next_token_dev, argmax_out_dev, B, K);
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

int adasd_gen_only_update(adasd_ctx* ctx, const float* H_draft_dev, const int32_t* draft_len_dev,
                          const int32_t* accept_len_dev, void* stream) {
    if (!ctx || !H_draft_dev || !accept_len_dev) return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned4({H_draft_dev, draft_len_dev, accept_len_dev})) return ADASD_ERR_ALIGN;
    const int B = ctx->cfg.B;
    gen_only_update_kernel<<<(B + 127) / 128, 128, 0, (cudaStream_t)stream>>>(ctx->st, H_draft_dev, draft_len_dev,
                                                                             accept_len_dev, B, ctx->cfg.Kmax);
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

int adasd_set_warpers(adasd_ctx* ctx, float temperature, int32_t top_k, float top_p) {
    if (!ctx) return ADASD_ERR_NULL;
    if (!(temperature > 0.f) || !std::isfinite(temperature)) return ADASD_ERR_SHAPE;
    if (!(top_p > 0.f) || top_p > 1.f) return ADASD_ERR_SHAPE;
    ctx->temperature = temperature;
    ctx->top_k = top_k < 0 ? 0 : top_k;
    ctx->top_p = top_p;
    return ADASD_OK;
}

int adasd_get_thresholds(adasd_ctx* ctx, float* T_G_dev, int32_t* nE_dev, int32_t* nA_dev,
                         int32_t* nR_dev, void* stream) {
    if (!ctx) return ADASD_ERR_NULL;
    if (int rc = check_device(ctx)) return rc;
    if (!aligned4({T_G_dev, nE_dev, nA_dev, nR_dev})) return ADASD_ERR_ALIGN;
    const int B = ctx->cfg.B;
    get_thresholds_kernel<<<(B + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
        ctx->st, T_G_dev, nE_dev, nA_dev, nR_dev, B);
    CUDA_TRY(cudaGetLastError());
    return ADASD_OK;
}

int adasd_state_export(adasd_ctx* ctx, int32_t seq, void* host_buf, size_t* bytes) {
    if (!ctx || !bytes) return ADASD_ERR_NULL;
    if (seq < 0 || seq >= ctx->cfg.B) return ADASD_ERR_SHAPE;
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(cudaDeviceSynchronize());
    const State& s = ctx->st;
    int32_t n[3];
    float tg;
    CUDA_TRY(cudaMemcpy(&n[0], s.nE + seq, 4, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemcpy(&n[1], s.nA + seq, 4, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemcpy(&n[2], s.nR + seq, 4, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemcpy(&tg, s.T_G + seq, 4, cudaMemcpyDeviceToHost));
    if (n[0] > s.cap) n[0] = s.cap;   // entropies beyond the capacity were only summed
    const size_t need = kExportHeader + 4 * ((size_t)n[0] + n[1] + n[2]);
    if (!host_buf) {
        *bytes = need;
        return ADASD_OK;
    }
    if (*bytes < need) {
        *bytes = need;
        return ADASD_ERR_CAPACITY;
    }
    char* o = static_cast<char*>(host_buf);
    int32_t hdr[4] = {n[0], n[1], n[2], 0};
    float fh[2] = {tg, 0.f};
    memcpy(o, hdr, 16);
    memcpy(o + 16, fh, 8);
    o += kExportHeader;
    const float* lists[3] = {s.LE, s.LA, s.LR};
    for (int k = 0; k < 3; ++k) {
        if (n[k] > 0)
            CUDA_TRY(cudaMemcpy(o, lists[k] + (size_t)seq * s.cap, 4 * (size_t)n[k],
                                cudaMemcpyDeviceToHost));
        o += 4 * (size_t)n[k];
    }
    *bytes = need;
    return ADASD_OK;
}

int adasd_state_import(adasd_ctx* ctx, int32_t seq, const void* host_buf, size_t bytes) {
    if (!ctx || !host_buf) return ADASD_ERR_NULL;
    if (seq < 0 || seq >= ctx->cfg.B || bytes < kExportHeader) return ADASD_ERR_SHAPE;
    const char* in = static_cast<const char*>(host_buf);
    int32_t hdr[4];
    float fh[2];
    memcpy(hdr, in, 16);
    memcpy(fh, in + 16, 8);
    const State& s = ctx->st;
    for (int k = 0; k < 3; ++k)
        if (hdr[k] < 0 || hdr[k] > s.cap) return ADASD_ERR_CAPACITY;
    if (bytes < kExportHeader + 4 * ((size_t)hdr[0] + hdr[1] + hdr[2])) return ADASD_ERR_SHAPE;
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(cudaDeviceSynchronize());
    const float* src = reinterpret_cast<const float*>(in + kExportHeader);
    float* lists[3] = {s.LE, s.LA, s.LR};
    double sums[3] = {0, 0, 0}, sums2[3] = {0, 0, 0};
    for (int k = 0; k < 3; ++k) {
        for (int j = 0; j < hdr[k]; ++j) {
            float v;
            memcpy(&v, src + j, 4);
            sums[k] += (double)v;
            sums2[k] += (double)v * (double)v;
        }
        if (hdr[k] > 0)
            CUDA_TRY(cudaMemcpy(lists[k] + (size_t)seq * s.cap, src, 4 * (size_t)hdr[k],
                                cudaMemcpyHostToDevice));
        src += hdr[k];
    }
    float tg = hdr[0] > 0 ? (float)(sums[0] / (double)hdr[0]) : fh[0];
    CUDA_TRY(cudaMemcpy(s.nE + seq, &hdr[0], 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.nA + seq, &hdr[1], 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.nR + seq, &hdr[2], 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.T_G + seq, &tg, 4, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.sumE + seq, &sums[0], 8, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.sumA + seq, &sums[1], 8, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.sumA2 + seq, &sums2[1], 8, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.sumR + seq, &sums[2], 8, cudaMemcpyHostToDevice));
    CUDA_TRY(cudaMemcpy(s.sumR2 + seq, &sums2[2], 8, cudaMemcpyHostToDevice));
    return ADASD_OK;
}

int adasd_status(adasd_ctx* ctx, uint32_t* status_out) {
    if (!ctx || !status_out) return ADASD_ERR_NULL;
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(status_out, ctx->st.status, 4, cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemset(ctx->st.status, 0, 4));
    return ADASD_OK;
}

int adasd_vanilla_verify_static(int32_t B, int32_t V, int32_t Kmax, int32_t dtype,
                                const void* draft_logits_dev, const void* target_logits_dev,
                                int64_t d_seq_stride, int64_t d_row_stride, int64_t t_seq_stride,
                                int64_t t_row_stride, const int32_t* draft_tokens_dev,
                                const int32_t* draft_len_dev, const float* u_accept_dev,
                                const float* u_resample_dev, int32_t* accept_len_dev,
                                int32_t* next_token_dev, float* alpha_out_dev,
                                uint32_t* status_out_dev, void* stream) {
    if (!draft_logits_dev || !target_logits_dev || !draft_tokens_dev || !u_accept_dev ||
        !u_resample_dev || !accept_len_dev || !next_token_dev)
        return ADASD_ERR_NULL;
    if (dtype != ADASD_BF16 && dtype != ADASD_FP32) return ADASD_ERR_DTYPE;
    if (B < 1 || V < 1 || Kmax < 1 || Kmax > ADASD_KMAX_LIMIT) return ADASD_ERR_SHAPE;
    if (B > ADASD_STATIC_MAX_B || (long long)B * (Kmax + 1) > ADASD_STATIC_MAX_POSITIONS)
        return ADASD_ERR_CAPACITY;
    if (d_row_stride < V || t_row_stride < V || d_seq_stride < 0 || t_seq_stride < 0)
        return ADASD_ERR_SHAPE;
    if (!aligned_to(draft_logits_dev, elt_size(dtype)) || !aligned_to(target_logits_dev, elt_size(dtype)) ||
        !aligned4({draft_tokens_dev, draft_len_dev, u_accept_dev, u_resample_dev, accept_len_dev,
                   next_token_dev, alpha_out_dev, status_out_dev}))
        return ADASD_ERR_ALIGN;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return ADASD_ERR_CUDA;
    }
    StaticSetup su;
    int rc = static_setup(dev, su);
    if (rc != ADASD_OK) return rc;

    cudaStream_t st = (cudaStream_t)stream;
    uint32_t* flag = su.base;
    uint32_t* tok = su.base + ADASD_STATIC_MAX_POSITIONS;
    uint32_t* ticket = su.base + 2 * ADASD_STATIC_MAX_POSITIONS;
    uint32_t* status = status_out_dev ? status_out_dev : ticket + ADASD_STATIC_MAX_B;
    // the array keeps whatever the previous call left: counters and status start at zero
    CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(uint32_t) * (size_t)B, st));
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(uint32_t), st));

    VerifyParams p;
    memset(&p, 0, sizeof(p));
    p.inv_temp = 1.f;                        // no context, no adjusted distribution
    p.c1 = kLog2e;
    p.zd = draft_logits_dev;
    p.zt = target_logits_dev;
    p.d_seq = d_seq_stride;
    p.d_row = d_row_stride;
    p.t_seq = t_seq_stride;
    p.t_row = t_row_stride;
    p.x = draft_tokens_dev;
    p.draft_len = draft_len_dev;
    p.u_accept = u_accept_dev;
    p.u_resample = u_resample_dev;
    p.accept_len = accept_len_dev;
    p.next_token = next_token_dev;
    p.alpha_out = alpha_out_dev;
    p.sc.van_flag = reinterpret_cast<int32_t*>(flag);
    p.sc.van_tok = reinterpret_cast<int32_t*>(tok);
    p.sc.ticket = ticket;
    p.st.status = status;
    p.B = B;
    p.V = V;
    p.Kmax = Kmax;
    p.tail.Kmax = Kmax;

    const long long positions = (long long)B * (Kmax + 1);
    int cs = kMaxCluster;
    for (int c = 1; c <= kMaxCluster; c *= 2)
        if (positions * c >= 2LL * su.sm_count) {
            cs = c;
            break;
        }
    const bool vec = vec_ok(draft_logits_dev, dtype, {d_seq_stride, d_row_stride}) &&
                     vec_ok(target_logits_dev, dtype, {t_seq_stride, t_row_stride});
    if (dtype == ADASD_BF16)
        return vec ? launch_cluster(verify_kernel<__nv_bfloat16, true, MODE_VANILLA>, p, positions, cs, st)
                   : launch_cluster(verify_kernel<__nv_bfloat16, false, MODE_VANILLA>, p, positions, cs, st);
    return vec ? launch_cluster(verify_kernel<float, true, MODE_VANILLA>, p, positions, cs, st)
               : launch_cluster(verify_kernel<float, false, MODE_VANILLA>, p, positions, cs, st);
}

const char* adasd_strerror(int code) {
    switch (code) {
        case ADASD_OK: return "ok";
        case ADASD_ERR_NULL: return "a required pointer is NULL";
        case ADASD_ERR_ALIGN: return "a pointer is not aligned to its element type";
        case ADASD_ERR_SHAPE: return "size, stride or window out of range";
        case ADASD_ERR_DTYPE: return "unknown dtype or rule";
        case ADASD_ERR_CAPACITY: return "size beyond a stated maximum";
        case ADASD_ERR_CUDA: return "a CUDA runtime call failed";
        case ADASD_ERR_DEVICE: return "the current device is not the context's device";
        default: return "unknown error";
    }
}

}  // extern "C"
