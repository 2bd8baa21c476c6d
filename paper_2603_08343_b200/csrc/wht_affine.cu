// C ABI of the library (see include/wht_affine.h): argument checks, kernel
// selection, launch geometry and the library-owned backward scratch buffer.
#include "../../include/wht_affine.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "bfly_kernels.cuh"
#include "mma_kernels.cuh"
#include "mma_pipe_kernels.cuh"
#include "tp_kernels.cuh"
#include "umma_kernels.cuh"

namespace {

using namespace wht;

constexpr int kMaxDevices = 64;
thread_local int g_last_cuda_error = 0;
int g_variant = 0;

struct DeviceState {
    int sm_count = 0;
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return WHT_ERR_CUDA;
}

// A kernel of which not even one CTA fits on an SM: report the runtime's error if it raised one,
// else "launch out of resources", so that WHT_ERR_CUDA never comes with a last-error of 0.
int occupancy_fail() {
    const cudaError_t e = cudaGetLastError();
    return cuda_fail(e != cudaSuccess ? e : cudaErrorLaunchOutOfResources);
}

#define WHT_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return cuda_fail(e__);       \
    } while (0)

int current_device(int* dev, int* sms) {
    WHT_CUDA_TRY(cudaGetDevice(dev));
    if (*dev < 0 || *dev >= kMaxDevices) return WHT_ERR_CUDA;
    DeviceState& st = g_dev[*dev];
    if (st.sm_count == 0) {
        int n = 0;
        WHT_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, *dev));
        st.sm_count = n;
    }
    *sms = st.sm_count;
    return WHT_OK;
}

bool is_pow2(int32_t d) { return d > 0 && (d & (d - 1)) == 0; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
int log2_of(int32_t d) { int l = 0; while ((1 << l) < d) ++l; return l; }
long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }

int check_common(int64_t T, int32_t d, int dtype) {
    if (dtype != WHT_F32 && dtype != WHT_BF16 && dtype != WHT_BF16_PF32) return WHT_ERR_BAD_DTYPE;
    if (!is_pow2(d) || d < 8 || d > 32768) return WHT_ERR_BAD_DIM;
    if (T < 0) return WHT_ERR_BAD_T;
    return WHT_OK;
}

// Resident CTAs per SM of one kernel instantiation, computed once per device.
template <typename Kernel>
int resident_ctas(Kernel kernel, int threads, size_t smem, int dev, int* cache) {
    if (cache[dev] > 0) return cache[dev];
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return 0;
    }
    if (smem > 0) {
        // first see how many CTAs fit when shared memory takes all it may ...
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared) != cudaSuccess)
            return 0;
    }
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess) return 0;
    if (smem > 0 && n > 0) {
        // ... then ask for no more than those CTAs need, so that what is left stays L1
        // (the per-channel parameters are re-read from L1 for every row)
        int max_smem_sm = 0;
        if (cudaDeviceGetAttribute(&max_smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess)
            return 0;
        const size_t want = static_cast<size_t>(n) * (smem + 1024);
        int pct = static_cast<int>((want * 100 + max_smem_sm - 1) / max_smem_sm);
        if (pct > 100) pct = 100;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, pct) != cudaSuccess)
            return 0;
        int n2 = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n2, kernel, threads, smem) != cudaSuccess) return 0;
        if (n2 < n) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                     cudaSharedmemCarveoutMaxShared) != cudaSuccess)
                return 0;
        }
    }
    cache[dev] = n > 0 ? n : 0;
    return cache[dev];
}

// Launch with the programmatic-stream-serialization attribute: the kernel may be scheduled
// while its predecessor in the stream drains.  Only for kernels that call
// grid_dependency_wait() before they touch global memory.
template <typename... KArgs, typename... Args>
void launch_overlapped(void (*kernel)(KArgs...), dim3 grid, int block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);  // errors are read by the caller (cudaGetLastError)
}

float inv_sqrt(int d) { return static_cast<float>(1.0 / sqrt(static_cast<double>(d))); }

// Everything a launcher needs besides the tensors.
struct Ctx {
    int64_t T;
    int dev;
    int sms;
    cudaStream_t stream;
    int64_t ld = 0;  // elements between consecutive rows; 0 = contiguous rows (ld == d)
    int groups = 1;  // block-diagonal form: channel groups of d side by side in a row (butterfly family only)
};

struct FwdArgs {
    const void* x;
    const void* a;
    const void* b;
    void* y;
    const void* resid = nullptr;  // fused residual input (layout and type of x), or none
};

struct BwdArgs {
    const void* dy;
    const void* x;
    const void* a;
    void* dx;
    float* da;
    float* db;
    void* ws;
    size_t ws_bytes;
    bool query_only;  // only report the scratch size in *need
    size_t* need;
};

// da = scale * (sum of the partials' first slots), db = sum of their second slots
int launch_finalize(const float* parts, int nparts, int d, float scale, float* da, float* db, cudaStream_t s) {
    if (d >= 32) {
        launch_overlapped(dadb_finalize32_kernel, 2 * d / 32, 1024, 0, s, parts, nparts, d, scale, da, db);
    } else {
        launch_overlapped(dadb_finalize_kernel, (2 * d + 255) / 256, 256, 0, s, parts, nparts, d, scale, da, db);
    }
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

// Common tail of every backward launcher: size the scratch, check it, launch, then the second pass
// (one per channel group; `grid` is the CTA count per group).
template <typename Launch>
int run_bwd_with_grid(const BwdArgs& g, const Ctx& c, int grid, int d, Launch launch, float scale = 0.0f) {
    *g.need = static_cast<size_t>(grid) * c.groups * 2 * d * sizeof(float);
    if (g.query_only) return WHT_OK;
    if (*g.need > 0 && (g.ws == nullptr || g.ws_bytes < *g.need)) return WHT_ERR_WORKSPACE;
    if (grid > 0) {
        launch(grid);
        WHT_CUDA_TRY(cudaGetLastError());
    }
    for (int grp = 0; grp < c.groups; ++grp) {
        const int rc = launch_finalize(static_cast<const float*>(g.ws) + static_cast<size_t>(grp) * grid * 2 * d, grid, d,
                                       scale > 0.0f ? scale : inv_sqrt(d), g.da + static_cast<size_t>(grp) * d,
                                       g.db + static_cast<size_t>(grp) * d, c.stream);
        if (rc != WHT_OK) return rc;
    }
    return WHT_OK;
}

int capped_grid(int64_t tiles, int sms, int per_sm) {
    const long long cap = static_cast<long long>(sms) * per_sm;
    return static_cast<int>(tiles < cap ? tiles : cap);
}

// ------------------------------------------------------------------ butterfly family
template <int LOGD, typename TIO, typename TP>
int launch_bfly_fwd(const FwdArgs& f, const Ctx& c) {
    using Geo = BflyFwdGeo<LOGD>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_fwd_kernel<LOGD, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    int grid = capped_grid(ceil_div(c.T, Geo::R), c.sms, per_sm);
    if (c.groups > 1) grid = grid / c.groups > 0 ? grid / c.groups : 1;  // CTAs per channel group
    launch_overlapped(kernel, dim3(grid, c.groups), Geo::THREADS, Geo::SMEM_FWD, c.stream,
                      static_cast<const TIO*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const TIO*>(f.resid), static_cast<TIO*>(f.y), static_cast<long long>(c.T),
                      static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, typename TIO, typename TP>
int launch_bfly_bwd(const BwdArgs& g, const Ctx& c) {
    using Geo = BflyBwdGeo<LOGD>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_bwd_kernel<LOGD, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    int grid = capped_grid(ceil_div(c.T, Geo::R), c.sms, per_sm);
    if (c.groups > 1) grid = grid / c.groups > 0 ? grid / c.groups : 1;  // CTAs per channel group
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        launch_overlapped(kernel, dim3(n, c.groups), Geo::THREADS, Geo::SMEM_BWD, c.stream,
                          static_cast<const TIO*>(g.dy), static_cast<const TIO*>(g.x), static_cast<const TP*>(g.a),
                          static_cast<TIO*>(g.dx), static_cast<float*>(g.ws), static_cast<long long>(c.T),
                          static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    });
}

#define WHT_FOR_EACH_LOGD(M) \
    M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)

template <typename TIO, typename TP>
int dispatch_bfly_fwd(int logd, const FwdArgs& f, const Ctx& c) {
    switch (logd) {
#define M(L) case L: return launch_bfly_fwd<L, TIO, TP>(f, c);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TIO, typename TP>
int dispatch_bfly_bwd(int logd, const BwdArgs& g, const Ctx& c) {
    switch (logd) {
#define M(L) case L: return launch_bfly_bwd<L, TIO, TP>(g, c);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

// ------------------------------------------------------------------ tensor-core family, direct loads
template <int LOGD, int TB, int RG, typename TP>
int launch_mma_fwd(const FwdArgs& f, const Ctx& c) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_fwd_kernel<LOGD, TB, RG, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, RG), c.sms, per_sm);
    launch_overlapped(kernel, grid, Geo::THREADS, Geo::SMEM_FWD, c.stream,
                      static_cast<const __nv_bfloat16*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const __nv_bfloat16*>(f.resid), static_cast<__nv_bfloat16*>(f.y),
                      static_cast<long long>(c.T), inv_sqrt(Geo::D));
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int TB, int RG, typename TP>
int launch_mma_bwd(const BwdArgs& g, const Ctx& c) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_bwd_kernel<LOGD, TB, RG, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, RG), c.sms, per_sm);
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        kernel<<<n, Geo::THREADS, Geo::SMEM_BWD, c.stream>>>(
            static_cast<const __nv_bfloat16*>(g.dy), static_cast<const __nv_bfloat16*>(g.x),
            static_cast<const TP*>(g.a), static_cast<__nv_bfloat16*>(g.dx), static_cast<float*>(g.ws),
            static_cast<long long>(c.T), inv_sqrt(Geo::D));
    });
}

// ------------------------------------------------------------------ tensor-core family, streamed rows
template <int LOGD, int TB, int RG, int S, int MINB, typename TP>
int launch_mma_fwd_pipe(const FwdArgs& f, const Ctx& c) {
    using Geo = PipeGeo<LOGD, TB, RG, S, false>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_fwd_pipe_kernel<LOGD, TB, RG, S, MINB, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, RG), c.sms, per_sm);
    kernel<<<grid, Geo::THREADS, Geo::SMEM, c.stream>>>(
        static_cast<const __nv_bfloat16*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
        static_cast<const __nv_bfloat16*>(f.resid), static_cast<__nv_bfloat16*>(f.y), static_cast<long long>(c.T),
        inv_sqrt(Geo::D));
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int TB, int RG, int S, int MINB, typename TP>
int launch_mma_bwd_pipe(const BwdArgs& g, const Ctx& c) {
    using Geo = PipeGeo<LOGD, TB, RG, S, true>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_bwd_pipe_kernel<LOGD, TB, RG, S, MINB, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, RG), c.sms, per_sm);
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        kernel<<<n, Geo::THREADS, Geo::SMEM, c.stream>>>(
            static_cast<const __nv_bfloat16*>(g.dy), static_cast<const __nv_bfloat16*>(g.x),
            static_cast<const TP*>(g.a), static_cast<__nv_bfloat16*>(g.dx), static_cast<float*>(g.ws),
            static_cast<long long>(c.T), inv_sqrt(Geo::D));
    });
}

// How a row is split for each d: (TB = log2 chunks per thread, RG = rows in flight
// per CTA, S = ring depth).  `few_rows` picks the direct-load kernels with a row
// spread over more warps (lowest latency per row: decode and small batches).
template <typename TP>
int dispatch_mma_fwd(int logd, bool few_rows, bool streamed, const FwdArgs& f, const Ctx& c) {
    if (few_rows) {
        switch (logd) {
            case 9: return launch_mma_fwd<9, 1, 4, TP>(f, c);
            case 10: return launch_mma_fwd<10, 1, 2, TP>(f, c);
            case 11: return launch_mma_fwd<11, 2, 2, TP>(f, c);
            // one row per CTA while every row gets an SM of its own, two beyond that
            case 12: return c.T > c.sms ? launch_mma_fwd<12, 2, 2, TP>(f, c) : launch_mma_fwd<12, 2, 1, TP>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, TP>(f, c);
        }
    } else if (!streamed) {
        switch (logd) {
            case 9: return launch_mma_fwd<9, 1, 4, TP>(f, c);
            case 10: return launch_mma_fwd<10, 2, 4, TP>(f, c);
            case 11: return launch_mma_fwd<11, 3, 4, TP>(f, c);
            case 12: return launch_mma_fwd<12, 3, 2, TP>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, TP>(f, c);
        }
    } else {
        switch (logd) {
            case 9: return launch_mma_fwd_pipe<9, 1, 8, 4, 2, TP>(f, c);
            case 10: return launch_mma_fwd_pipe<10, 2, 8, 4, 3, TP>(f, c);
            case 11: return launch_mma_fwd_pipe<11, 3, 8, 3, 2, TP>(f, c);
            case 12: return launch_mma_fwd_pipe<12, 3, 2, 3, 2, TP>(f, c);
            case 13: return launch_mma_fwd_pipe<13, 3, 2, 2, 1, TP>(f, c);
        }
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TP>
int dispatch_mma_bwd(int logd, bool streamed, const BwdArgs& g, const Ctx& c) {
    if (!streamed) {
        switch (logd) {
            case 9: return launch_mma_bwd<9, 1, 8, TP>(g, c);
            case 10: return launch_mma_bwd<10, 2, 8, TP>(g, c);
            case 11: return launch_mma_bwd<11, 2, 4, TP>(g, c);
            case 12: return launch_mma_bwd<12, 2, 2, TP>(g, c);
            case 13: return launch_mma_bwd<13, 3, 1, TP>(g, c);
        }
    } else {
        switch (logd) {
            case 9: return launch_mma_bwd_pipe<9, 1, 8, 4, 2, TP>(g, c);
            case 10: return launch_mma_bwd_pipe<10, 2, 8, 3, 2, TP>(g, c);
            case 11: return launch_mma_bwd_pipe<11, 2, 4, 2, 2, TP>(g, c);
            case 12: return launch_mma_bwd_pipe<12, 2, 2, 2, 1, TP>(g, c);
            case 13: return launch_mma_bwd_pipe<13, 3, 1, 2, 1, TP>(g, c);
        }
    }
    return WHT_ERR_BAD_DIM;
}

// ------------------------------------------------------------------ tcgen05 family
// One persistent CTA per SM; a kernel's shared-memory need alone keeps a second CTA off the SM,
// which the kernel relies on when it allocates tensor memory.
template <typename Kernel>
int prepare_umma(Kernel kernel, int smem, int dev, int* cache) {
    if (cache[dev]) return WHT_OK;
    WHT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cache[dev] = 1;
    return WHT_OK;
}

template <int LOGD, int NCOL, int STAGES, typename TP, bool RES>
int launch_umma_fwd_impl(const FwdArgs& f, const Ctx& c) {
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaFwdSmem<LOGD, NCOL, STAGES, TP, RES>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_fwd_kernel<LOGD, NCOL, STAGES, TP, RES>;
    int rc = prepare_umma(kernel, L::BYTES, c.dev, ready);
    if (rc != WHT_OK) return rc;
    const int grid = capped_grid(ceil_div(c.T, Geo::ROWS), c.sms, 1);
    launch_overlapped(kernel, grid, Geo::THREADS, L::BYTES, c.stream,
                      static_cast<const __nv_bfloat16*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const __nv_bfloat16*>(f.resid), static_cast<__nv_bfloat16*>(f.y),
                      static_cast<long long>(c.T), inv_sqrt(Geo::D), TpParts{}, 1, 0u);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int NCOL, int STAGES, typename TP>
int launch_umma_fwd(const FwdArgs& f, const Ctx& c) {
    return f.resid ? launch_umma_fwd_impl<LOGD, NCOL, STAGES, TP, true>(f, c)
                   : launch_umma_fwd_impl<LOGD, NCOL, STAGES, TP, false>(f, c);
}

template <int LOGD, int NCOL, int STAGES, typename TP, bool A_TMEM>
int launch_umma_bwd_impl(const BwdArgs& g, const Ctx& c) {
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaBwdSmem<LOGD, NCOL, STAGES>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_bwd_kernel<LOGD, NCOL, STAGES, TP, A_TMEM>;
    if (!g.query_only) {
        int rc = prepare_umma(kernel, L::BYTES, c.dev, ready);
        if (rc != WHT_OK) return rc;
    }
    const int grid = capped_grid(ceil_div(c.T, Geo::ROWS), c.sms, 1);
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        launch_overlapped(kernel, n, Geo::THREADS, L::BYTES, c.stream,
                          static_cast<const __nv_bfloat16*>(g.dy), static_cast<const __nv_bfloat16*>(g.x),
                          static_cast<const TP*>(g.a), static_cast<__nv_bfloat16*>(g.dx), static_cast<float*>(g.ws),
                          static_cast<long long>(c.T), inv_sqrt(Geo::D));
    });
}

// H_128 in tensor memory: in long runs under the power cap measured 4 % faster than the shared-memory
// operand at d = 8192 and 0-1 % at d = 2048 (less shared-memory traffic per product), the same in short bursts.
template <int LOGD, int NCOL, int STAGES, typename TP>
int launch_umma_bwd(const BwdArgs& g, const Ctx& c) {
    return launch_umma_bwd_impl<LOGD, NCOL, STAGES, TP, true>(g, c);
}

template <typename TP>
int dispatch_umma_fwd(int logd, const FwdArgs& f, const Ctx& c) {
    switch (logd) {
        case 10: return launch_umma_fwd<10, 128, 4, TP>(f, c);
        case 11: return launch_umma_fwd<11, 128, 4, TP>(f, c);
        case 12: return launch_umma_fwd<12, 128, 4, TP>(f, c);
        case 13: return launch_umma_fwd<13, 128, 4, TP>(f, c);
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TP>
int dispatch_umma_bwd(int logd, const BwdArgs& g, const Ctx& c) {
    switch (logd) {
        case 10: return launch_umma_bwd<10, 128, 3, TP>(g, c);
        case 11: return launch_umma_bwd<11, 128, 3, TP>(g, c);
        case 12: return launch_umma_bwd<12, 128, 3, TP>(g, c);
        case 13: return launch_umma_bwd<13, 128, 3, TP>(g, c);
    }
    return WHT_ERR_BAD_DIM;
}

bool umma_fwd_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 10 && logd <= 13; }
bool umma_bwd_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 10 && logd <= 13; }

bool mma_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 9 && logd <= 13; }

// The persistent tcgen05 kernels win once there are a few hundred 32 KiB tiles (measured
// cross-over against the direct-load kernels, CUDA-graph replay, d = 1024 ... 8192).
bool enough_work_for_tiles(int64_t T, int32_t d) {
    const int64_t elems = T * static_cast<int64_t>(d);
    return elems >= (d >= 8192 ? (8ll << 20) : (4ll << 20));
}

// Streaming pays once every row group has several rows to pipeline.
bool enough_rows_to_stream(int64_t T, int sms) { return T >= static_cast<int64_t>(sms) * 32; }

// ------------------------------------------------------------------ selection
int run_fwd(const FwdArgs& f, int64_t T, int32_t d, int dtype, cudaStream_t s, bool decode) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    const int logd = log2_of(d);
    if (umma_fwd_supported(logd, dtype) &&
        (g_variant == 4 || (g_variant == 0 && enough_work_for_tiles(T, d)))) {
        return dtype == WHT_BF16 ? dispatch_umma_fwd<__nv_bfloat16>(logd, f, c) : dispatch_umma_fwd<float>(logd, f, c);
    }
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        const bool streamed = g_variant >= 3 || (g_variant == 0 && !decode && enough_rows_to_stream(T, c.sms));
        const bool few_rows = !streamed && (decode || (g_variant == 0 && T < static_cast<int64_t>(c.sms) * 4));
        return dtype == WHT_BF16 ? dispatch_mma_fwd<__nv_bfloat16>(logd, few_rows, streamed, f, c)
                                 : dispatch_mma_fwd<float>(logd, few_rows, streamed, f, c);
    }
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_fwd<float, float>(logd, f, c);
        case WHT_BF16: return dispatch_bfly_fwd<__nv_bfloat16, __nv_bfloat16>(logd, f, c);
        default: return dispatch_bfly_fwd<__nv_bfloat16, float>(logd, f, c);
    }
}

int run_bwd(const BwdArgs& g, int64_t T, int32_t d, int dtype, cudaStream_t s) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    const int logd = log2_of(d);
    // the backward is the heavier kernel: the tcgen05 form was never slower than the others from a
    // few hundred rows on
    if (umma_bwd_supported(logd, dtype) &&
        (g_variant == 4 || (g_variant == 0 && T * static_cast<int64_t>(d) >= (1ll << 18)))) {
        return dtype == WHT_BF16 ? dispatch_umma_bwd<__nv_bfloat16>(logd, g, c) : dispatch_umma_bwd<float>(logd, g, c);
    }
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        const bool streamed = g_variant >= 3 || (g_variant == 0 && enough_rows_to_stream(T, c.sms));
        return dtype == WHT_BF16 ? dispatch_mma_bwd<__nv_bfloat16>(logd, streamed, g, c)
                                 : dispatch_mma_bwd<float>(logd, streamed, g, c);
    }
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_bwd<float, float>(logd, g, c);
        case WHT_BF16: return dispatch_bfly_bwd<__nv_bfloat16, __nv_bfloat16>(logd, g, c);
        default: return dispatch_bfly_bwd<__nv_bfloat16, float>(logd, g, c);
    }
}

int check_fwd_args(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d, int dtype) {
    int rc = check_common(T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (!a || !b) return WHT_ERR_NULL;
    if (T > 0 && (!x || !y)) return WHT_ERR_NULL;  // empty row tensors may have no storage
    if (!aligned16(x) || !aligned16(a) || !aligned16(b) || !aligned16(y)) return WHT_ERR_MISALIGNED;
    return WHT_OK;
}

int check_bwd_args(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                   int64_t T, int32_t d, int dtype) {
    int rc = check_common(T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (!a || !da || !db) return WHT_ERR_NULL;
    if (T > 0 && (!dy || !x || !dx)) return WHT_ERR_NULL;  // empty row tensors may have no storage
    if (!aligned16(dy) || !aligned16(x) || !aligned16(a) || !aligned16(dx) || !aligned16(da) || !aligned16(db))
        return WHT_ERR_MISALIGNED;
    return WHT_OK;
}

// Scratch of wht_affine_bwd_noalloc: part of the device image, so no call ever
// allocates it.  In host code this name is only a handle for the runtime -- the
// device address comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[WHT_NOALLOC_SCRATCH_BYTES];
void* g_noalloc_scratch_ptr[kMaxDevices] = {};

int noalloc_scratch_for_current_device(int dev, void** out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_noalloc_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        WHT_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));  // address on the CURRENT device
        if (p == nullptr) return WHT_ERR_WORKSPACE;
        g_noalloc_scratch_ptr[dev] = p;
    }
    *out = g_noalloc_scratch_ptr[dev];
    return WHT_OK;
}

// ------------------------------------------------------------------ column-sharded (tensor-parallel) form
struct TpCall {
    TpParts xs;       // the g blocks of x (this rank's own and the peers')
    TpParts dys;      // backward only
    TpParts as;       // backward only: every rank's a block
    int g;
    int r;
    unsigned neg_mask;  // bit s set: H_g[s][r] = -1
    float scale;        // 1/sqrt(g*w)
};

template <int LOGW, typename TIO, typename TP>
int launch_bfly_fwd_tp(const TpCall& t, const FwdArgs& f, const Ctx& c) {
    using Geo = BflyFwdGeo<LOGW>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_fwd_tp_kernel<LOGW, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, Geo::R), c.sms, per_sm);
    kernel<<<grid, Geo::THREADS, Geo::SMEM_FWD, c.stream>>>(t.xs, t.g, t.neg_mask, static_cast<const TP*>(f.a),
                                                            static_cast<const TP*>(f.b), static_cast<TIO*>(f.y),
                                                            static_cast<long long>(c.T), t.scale);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGW, typename TIO, typename TP>
int launch_bfly_bwd_tp(const TpCall& t, const BwdArgs& g, const Ctx& c) {
    using Geo = BflyBwdGeo<LOGW>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_bwd_tp_kernel<LOGW, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = capped_grid(ceil_div(c.T, Geo::R), c.sms, per_sm);
    return run_bwd_with_grid(
        g, c, grid, Geo::D,
        [&](int n) {
            kernel<<<n, Geo::THREADS, Geo::SMEM_BWD, c.stream>>>(t.dys, t.xs, t.as, t.g, t.r, t.neg_mask,
                                                                 static_cast<TIO*>(g.dx), static_cast<float*>(g.ws),
                                                                 static_cast<long long>(c.T), t.scale);
        },
        t.scale);
}

// tcgen05 form of the column-sharded forward: one product per source block into one accumulator
template <int LOGW, typename TP>
int launch_umma_fwd_tp(const TpCall& t, const FwdArgs& f, const Ctx& c) {
    constexpr int NCOL = 128, STAGES = 4;
    using Geo = UmmaGeo<LOGW, NCOL>;
    using L = UmmaFwdSmem<LOGW, NCOL, STAGES, TP, false>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static_assert(!L::SPLIT, "widths handled here keep every channel of a row in one thread group");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_fwd_kernel<LOGW, NCOL, STAGES, TP, false, true>;
    int rc = prepare_umma(kernel, L::BYTES, c.dev, ready);
    if (rc != WHT_OK) return rc;
    const int grid = capped_grid(ceil_div(c.T, Geo::ROWS), c.sms, 1);
    launch_overlapped(kernel, grid, Geo::THREADS, L::BYTES, c.stream, static_cast<const __nv_bfloat16*>(nullptr),
                      static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const __nv_bfloat16*>(nullptr), static_cast<__nv_bfloat16*>(f.y),
                      static_cast<long long>(c.T), t.scale, t.xs, t.g, t.neg_mask);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <typename TP>
int dispatch_umma_fwd_tp(int logw, const TpCall& t, const FwdArgs& f, const Ctx& c) {
    switch (logw) {
        case 10: return launch_umma_fwd_tp<10, TP>(t, f, c);
        case 11: return launch_umma_fwd_tp<11, TP>(t, f, c);
        case 12: return launch_umma_fwd_tp<12, TP>(t, f, c);
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TIO, typename TP>
int dispatch_bfly_fwd_tp(int logw, const TpCall& t, const FwdArgs& f, const Ctx& c) {
    switch (logw) {
#define M(L) case L: return launch_bfly_fwd_tp<L, TIO, TP>(t, f, c);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TIO, typename TP>
int dispatch_bfly_bwd_tp(int logw, const TpCall& t, const BwdArgs& g, const Ctx& c) {
    switch (logw) {
#define M(L) case L: return launch_bfly_bwd_tp<L, TIO, TP>(t, g, c);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

int check_tp(int64_t T, int32_t w, int32_t g, int32_t r, int dtype) {
    int rc = check_common(T, w, dtype);
    if (rc != WHT_OK) return rc;
    if (!is_pow2(g) || g > kTpMaxRanks || r < 0 || r >= g) return WHT_ERR_BAD_DIM;
    return WHT_OK;
}

// Copies g device pointers out of a host array, checking each.
int gather_parts(const void* const* parts, int g, bool need_data, TpParts* out) {
    if (!parts) return WHT_ERR_NULL;
    for (int s = 0; s < kTpMaxRanks; ++s) out->p[s] = nullptr;
    for (int s = 0; s < g; ++s) {
        if (need_data && !parts[s]) return WHT_ERR_NULL;
        if (!aligned16(parts[s])) return WHT_ERR_MISALIGNED;
        out->p[s] = parts[s];
    }
    return WHT_OK;
}

unsigned tp_neg_mask(int g, int r) {
    unsigned m = 0;
    for (int s = 0; s < g; ++s)
        if (__builtin_popcount(static_cast<unsigned>(s & r)) & 1) m |= 1u << s;
    return m;
}

int run_bwd_tp(const TpCall& t, const BwdArgs& g, int64_t T, int32_t w, int dtype, cudaStream_t s) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    const int logw = log2_of(w);
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_bwd_tp<float, float>(logw, t, g, c);
        case WHT_BF16: return dispatch_bfly_bwd_tp<__nv_bfloat16, __nv_bfloat16>(logw, t, g, c);
        default: return dispatch_bfly_bwd_tp<__nv_bfloat16, float>(logw, t, g, c);
    }
}

int query_bwd_bytes(int64_t T, int32_t d, int dtype, size_t* need) {
    BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, need};
    return run_bwd(q, T, d, dtype, nullptr);
}

}  // namespace

extern "C" {

int wht_affine_fwd(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d,
                   int dtype, void* stream) {
    int rc = check_fwd_args(x, a, b, y, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (T == 0) return WHT_OK;
    return run_fwd(FwdArgs{x, a, b, y}, T, d, dtype, static_cast<cudaStream_t>(stream), false);
}

int wht_affine_fwd_decode(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d,
                          int dtype, void* stream) {
    int rc = check_fwd_args(x, a, b, y, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (T == 0) return WHT_OK;
    return run_fwd(FwdArgs{x, a, b, y}, T, d, dtype, static_cast<cudaStream_t>(stream), true);
}

int wht_affine_fwd_residual(const void* x, const void* a, const void* b, const void* resid, void* y, int64_t T,
                            int32_t d, int dtype, void* stream) {
    int rc = check_fwd_args(x, a, b, y, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (T > 0 && !resid) return WHT_ERR_NULL;
    if (!aligned16(resid)) return WHT_ERR_MISALIGNED;
    if (T == 0) return WHT_OK;
    FwdArgs f{x, a, b, y};
    f.resid = resid;
    return run_fwd(f, T, d, dtype, static_cast<cudaStream_t>(stream), false);
}

size_t wht_affine_bwd_workspace_bytes(int64_t T, int32_t d, int dtype) {
    if (check_common(T, d, dtype) != WHT_OK) return 0;
    size_t need = 0;
    if (query_bwd_bytes(T, d, dtype, &need) != WHT_OK) return 0;
    return need;
}

int wht_affine_bwd_ws(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                      int64_t T, int32_t d, int dtype, void* workspace, size_t workspace_bytes,
                      void* stream) {
    int rc = check_bwd_args(dy, x, a, dx, da, db, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (workspace && !aligned16(workspace)) return WHT_ERR_MISALIGNED;
    size_t need = 0;
    BwdArgs g{dy, x, a, dx, da, db, workspace, workspace_bytes, false, &need};
    return run_bwd(g, T, d, dtype, static_cast<cudaStream_t>(stream));
}

int wht_affine_bwd(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                   int64_t T, int32_t d, int dtype, void* stream) {
    int rc = check_bwd_args(dy, x, a, dx, da, db, T, d, dtype);
    if (rc != WHT_OK) return rc;
    size_t need = 0;
    rc = query_bwd_bytes(T, d, dtype, &need);
    if (rc != WHT_OK) return rc;
    int dev = 0, sms = 0;
    rc = current_device(&dev, &sms);
    if (rc != WHT_OK) return rc;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        DeviceState& st = g_dev[dev];
        if (st.scratch_bytes < need) {
            // growing: wait for work that may still read the old buffer, then replace it
            if (st.scratch) {
                WHT_CUDA_TRY(cudaDeviceSynchronize());
                WHT_CUDA_TRY(cudaFree(st.scratch));
                st.scratch = nullptr;
                st.scratch_bytes = 0;
            }
            void* p = nullptr;
            const size_t bytes = need < (1u << 20) ? (1u << 20) : need;
            if (cudaMalloc(&p, bytes) != cudaSuccess) {
                g_last_cuda_error = static_cast<int>(cudaGetLastError());
                return WHT_ERR_WORKSPACE;
            }
            st.scratch = p;
            st.scratch_bytes = bytes;
        }
        ws = st.scratch;
        ws_bytes = st.scratch_bytes;
    }
    BwdArgs g{dy, x, a, dx, da, db, ws, ws_bytes, false, &need};
    return run_bwd(g, T, d, dtype, static_cast<cudaStream_t>(stream));
}

int wht_affine_bwd_noalloc(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                           int64_t T, int32_t d, int dtype, void* stream) {
    int rc = check_bwd_args(dy, x, a, dx, da, db, T, d, dtype);
    if (rc != WHT_OK) return rc;
    size_t need = 0;
    rc = query_bwd_bytes(T, d, dtype, &need);
    if (rc != WHT_OK) return rc;
    if (need > WHT_NOALLOC_SCRATCH_BYTES) return WHT_ERR_WORKSPACE;  // beyond the built-in array
    int dev = 0, sms = 0;
    rc = current_device(&dev, &sms);
    if (rc != WHT_OK) return rc;
    void* ws = nullptr;
    rc = noalloc_scratch_for_current_device(dev, &ws);
    if (rc != WHT_OK) return rc;
    BwdArgs g{dy, x, a, dx, da, db, ws, WHT_NOALLOC_SCRATCH_BYTES, false, &need};
    return run_bwd(g, T, d, dtype, static_cast<cudaStream_t>(stream));
}

// ---- grouped (block-diagonal) form: d = groups * block, every block transformed on its own.
// One launch of the butterfly family with the channel group as the grid's second dimension.
namespace {
int check_grouped(int64_t T, int32_t d, int32_t block, int dtype) {
    if (dtype != WHT_F32 && dtype != WHT_BF16 && dtype != WHT_BF16_PF32) return WHT_ERR_BAD_DTYPE;
    if (!is_pow2(block) || block < 8 || block > 32768 || d < block || d % block != 0) return WHT_ERR_BAD_DIM;
    if (T < 0) return WHT_ERR_BAD_T;
    return WHT_OK;
}
}  // namespace

int wht_affine_fwd_grouped(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d,
                           int32_t block, int dtype, void* stream) {
    int rc = check_grouped(T, d, block, dtype);
    if (rc != WHT_OK) return rc;
    if (!a || !b) return WHT_ERR_NULL;
    if (T > 0 && (!x || !y)) return WHT_ERR_NULL;
    if (!aligned16(x) || !aligned16(a) || !aligned16(b) || !aligned16(y)) return WHT_ERR_MISALIGNED;
    if (T == 0) return WHT_OK;
    Ctx c{T, 0, 0, static_cast<cudaStream_t>(stream)};
    c.ld = d;
    rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    c.groups = d / block;
    const int logb = log2_of(block);
    const FwdArgs f{x, a, b, y};
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_fwd<float, float>(logb, f, c);
        case WHT_BF16: return dispatch_bfly_fwd<__nv_bfloat16, __nv_bfloat16>(logb, f, c);
        default: return dispatch_bfly_fwd<__nv_bfloat16, float>(logb, f, c);
    }
}

int wht_affine_bwd_grouped(const void* dy, const void* x, const void* a, void* dx, float* da, float* db, int64_t T,
                           int32_t d, int32_t block, int dtype, void* workspace, size_t workspace_bytes,
                           void* stream) {
    int rc = check_grouped(T, d, block, dtype);
    if (rc != WHT_OK) return rc;
    if (!a || !da || !db) return WHT_ERR_NULL;
    if (T > 0 && (!dy || !x || !dx)) return WHT_ERR_NULL;
    if (!aligned16(dy) || !aligned16(x) || !aligned16(a) || !aligned16(dx) || !aligned16(da) || !aligned16(db) ||
        !aligned16(workspace))
        return WHT_ERR_MISALIGNED;
    Ctx c{T, 0, 0, static_cast<cudaStream_t>(stream)};
    c.ld = d;
    rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    c.groups = d / block;
    const int logb = log2_of(block);
    size_t need = 0;
    const BwdArgs q{dy, x, a, dx, da, db, workspace, workspace_bytes, false, &need};
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_bwd<float, float>(logb, q, c);
        case WHT_BF16: return dispatch_bfly_bwd<__nv_bfloat16, __nv_bfloat16>(logb, q, c);
        default: return dispatch_bfly_bwd<__nv_bfloat16, float>(logb, q, c);
    }
}

size_t wht_affine_bwd_grouped_workspace_bytes(int64_t T, int32_t d, int32_t block, int dtype) {
    if (check_grouped(T, d, block, dtype) != WHT_OK) return 0;
    Ctx c{T, 0, 0, nullptr};
    if (current_device(&c.dev, &c.sms) != WHT_OK) return 0;
    c.groups = d / block;
    size_t need = 0;
    BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, &need};
    int rc;
    switch (dtype) {
        case WHT_F32: rc = dispatch_bfly_bwd<float, float>(log2_of(block), q, c); break;
        case WHT_BF16: rc = dispatch_bfly_bwd<__nv_bfloat16, __nv_bfloat16>(log2_of(block), q, c); break;
        default: rc = dispatch_bfly_bwd<__nv_bfloat16, float>(log2_of(block), q, c); break;
    }
    return rc == WHT_OK ? need : 0;
}

// ---- column-sharded (tensor-parallel) form: see the header.
int wht_affine_fwd_tp(const void* const* x_parts, const void* a, const void* b, void* y, int64_t T, int32_t w,
                      int32_t g, int32_t r, int dtype, void* stream) {
    int rc = check_tp(T, w, g, r, dtype);
    if (rc != WHT_OK) return rc;
    if (!a || !b || (T > 0 && !y)) return WHT_ERR_NULL;
    if (!aligned16(a) || !aligned16(b) || !aligned16(y)) return WHT_ERR_MISALIGNED;
    TpCall t{};
    rc = gather_parts(x_parts, g, T > 0, &t.xs);
    if (rc != WHT_OK) return rc;
    if (T == 0) return WHT_OK;
    t.g = g;
    t.r = r;
    t.neg_mask = tp_neg_mask(g, r);
    t.scale = static_cast<float>(1.0 / sqrt(static_cast<double>(g) * w));
    Ctx c{T, 0, 0, static_cast<cudaStream_t>(stream)};
    rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    const FwdArgs f{nullptr, a, b, y};
    const int logw = log2_of(w);
    // bf16 rows of 1024 ... 4096 channels per rank with enough rows for 32 KiB tiles: tcgen05 form
    if (dtype != WHT_F32 && logw >= 10 && logw <= 12 && (g_variant == 0 || g_variant == 4) &&
        (g_variant == 4 || enough_work_for_tiles(T, w))) {
        return dtype == WHT_BF16 ? dispatch_umma_fwd_tp<__nv_bfloat16>(logw, t, f, c)
                                 : dispatch_umma_fwd_tp<float>(logw, t, f, c);
    }
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_fwd_tp<float, float>(logw, t, f, c);
        case WHT_BF16: return dispatch_bfly_fwd_tp<__nv_bfloat16, __nv_bfloat16>(logw, t, f, c);
        default: return dispatch_bfly_fwd_tp<__nv_bfloat16, float>(logw, t, f, c);
    }
}

size_t wht_affine_bwd_tp_workspace_bytes(int64_t T, int32_t w, int32_t g, int dtype) {
    if (check_tp(T, w, g, 0, dtype) != WHT_OK) return 0;
    size_t need = 0;
    BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, &need};
    TpCall t{};
    t.g = g;
    if (run_bwd_tp(t, q, T, w, dtype, nullptr) != WHT_OK) return 0;
    return need;
}

int wht_affine_bwd_tp(const void* const* dy_parts, const void* const* x_parts, const void* const* a_parts, void* dx,
                      float* da, float* db, int64_t T, int32_t w, int32_t g, int32_t r, int dtype, void* workspace,
                      size_t workspace_bytes, void* stream) {
    int rc = check_tp(T, w, g, r, dtype);
    if (rc != WHT_OK) return rc;
    if (!da || !db || (T > 0 && !dx)) return WHT_ERR_NULL;
    if (!aligned16(dx) || !aligned16(da) || !aligned16(db) || !aligned16(workspace)) return WHT_ERR_MISALIGNED;
    TpCall t{};
    rc = gather_parts(dy_parts, g, T > 0, &t.dys);
    if (rc == WHT_OK) rc = gather_parts(x_parts, g, T > 0, &t.xs);
    if (rc == WHT_OK) rc = gather_parts(a_parts, g, true, &t.as);
    if (rc != WHT_OK) return rc;
    t.g = g;
    t.r = r;
    t.neg_mask = tp_neg_mask(g, r);
    t.scale = static_cast<float>(1.0 / sqrt(static_cast<double>(g) * w));
    size_t need = 0;
    BwdArgs b{nullptr, nullptr, nullptr, dx, da, db, workspace, workspace_bytes, false, &need};
    return run_bwd_tp(t, b, T, w, dtype, static_cast<cudaStream_t>(stream));
}

int wht_affine_reduce_grads(const float* parts, int32_t n, int32_t d, float* da, float* db, void* stream) {
    if (!is_pow2(d) || d < 8 || d > 32768) return WHT_ERR_BAD_DIM;
    if (n < 0) return WHT_ERR_BAD_T;
    if (!da || !db || (n > 0 && !parts)) return WHT_ERR_NULL;
    if (!aligned16(parts) || !aligned16(da) || !aligned16(db)) return WHT_ERR_MISALIGNED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the second pass of the backward with a unit scale: partial p, slot 0 = da_p, slot 1 = db_p
    if (d >= 32) {
        launch_overlapped(dadb_finalize32_kernel, 2 * d / 32, 1024, 0, s, parts, static_cast<int>(n),
                          static_cast<int>(d), 1.0f, da, db);
    } else {
        launch_overlapped(dadb_finalize_kernel, (2 * d + 255) / 256, 256, 0, s, parts, static_cast<int>(n),
                          static_cast<int>(d), 1.0f, da, db);
    }
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

int wht_affine_set_variant(int variant) {
    if (variant < 0 || variant > 4) return WHT_ERR_BAD_VARIANT;
    g_variant = variant;
    return WHT_OK;
}

int wht_affine_get_variant(void) { return g_variant; }

int wht_copy_rows(const void* src, void* dst, int64_t T, int32_t d, int dtype, void* stream) {
    int rc = check_common(T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (!src || !dst) return WHT_ERR_NULL;
    if (!aligned16(src) || !aligned16(dst)) return WHT_ERR_MISALIGNED;
    if (T == 0) return WHT_OK;
    int dev = 0, sms = 0;
    rc = current_device(&dev, &sms);
    if (rc != WHT_OK) return rc;
    const long long elem = dtype == WHT_F32 ? 4 : 2;
    const long long n16 = static_cast<long long>(T) * d * elem / 16;
    copy_rows_kernel<<<capped_grid(ceil_div(n16, 256), sms, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), n16);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

int wht_affine_device_status(void) {
    unsigned int flag = 0;
    WHT_CUDA_TRY(cudaMemcpyFromSymbol(&flag, g_wht_device_error, sizeof(flag)));
    if (flag == 0) return WHT_OK;
    const unsigned int zero = 0;
    WHT_CUDA_TRY(cudaMemcpyToSymbol(g_wht_device_error, &zero, sizeof(zero)));
    return WHT_ERR_DEVICE_WAIT;
}

int wht_affine_last_cuda_error(void) { return g_last_cuda_error; }

const char* wht_affine_status_string(int status) {
    switch (status) {
        case WHT_OK: return "WHT_OK";
        case WHT_ERR_NULL: return "WHT_ERR_NULL: a required pointer is NULL";
        case WHT_ERR_BAD_DIM: return "WHT_ERR_BAD_DIM: d must be a power of two in [8, 32768]";
        case WHT_ERR_BAD_T: return "WHT_ERR_BAD_T: T must be >= 0";
        case WHT_ERR_BAD_DTYPE: return "WHT_ERR_BAD_DTYPE: unknown dtype code";
        case WHT_ERR_MISALIGNED: return "WHT_ERR_MISALIGNED: pointers must be 16-byte aligned";
        case WHT_ERR_WORKSPACE: return "WHT_ERR_WORKSPACE: scratch buffer missing, too small or not allocatable";
        case WHT_ERR_CUDA: return "WHT_ERR_CUDA: a CUDA runtime call failed";
        case WHT_ERR_BAD_VARIANT: return "WHT_ERR_BAD_VARIANT: unknown kernel variant";
        case WHT_ERR_DEVICE_WAIT:
            return "WHT_ERR_DEVICE_WAIT: a kernel gave up waiting for an async copy; that launch's results are invalid";
        default: return "unknown wht_status";
    }
}

int wht_affine_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int rc = WHT_OK;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    for (int dev = 0; dev < kMaxDevices; ++dev) {
        DeviceState& st = g_dev[dev];
        if (!st.scratch) continue;
        if (cudaSetDevice(dev) != cudaSuccess || cudaFree(st.scratch) != cudaSuccess) {
            g_last_cuda_error = static_cast<int>(cudaGetLastError());
            rc = WHT_ERR_CUDA;
        }
        st.scratch = nullptr;
        st.scratch_bytes = 0;
    }
    if (prev >= 0) cudaSetDevice(prev);
    return rc;
}

}  // extern "C"
