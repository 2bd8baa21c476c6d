// Host-side pieces shared by the translation units of the library: the C ABI and kernel selection
// (wht_affine.cu) and one file per kernel family (family_*.cu), each of which instantiates its own
// kernels and exports plain dispatch functions.  The split only exists so that the families compile
// in parallel; nothing here is visible outside the library.
#pragma once
#include "../../include/wht_affine.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstddef>
#include <cstdint>

#include "wht_common.cuh"

namespace wht_host {

constexpr int kMaxDevices = 64;

// error reporting (state lives in wht_affine.cu)
int cuda_fail(cudaError_t e);
// A kernel of which not even one CTA fits on an SM: reports the runtime's error if it raised one,
// else "launch out of resources", so that WHT_ERR_CUDA never comes with a last-error of 0.
int occupancy_fail();

#define WHT_CUDA_TRY(expr)                                        \
    do {                                                          \
        cudaError_t e__ = (expr);                                 \
        if (e__ != cudaSuccess) return ::wht_host::cuda_fail(e__); \
    } while (0)

inline int log2_of(int32_t d) { int l = 0; while ((1 << l) < d) ++l; return l; }
inline long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }
inline float inv_sqrt(int d) { return static_cast<float>(1.0 / std::sqrt(static_cast<double>(d))); }
inline int capped_grid(int64_t tiles, int sms, int per_sm) {
    const long long cap = static_cast<long long>(sms) * per_sm;
    return static_cast<int>(tiles < cap ? tiles : cap);
}

// Everything a launcher needs besides the tensors.
struct Ctx {
    int64_t T;
    int dev;
    int sms;
    cudaStream_t stream;
    int64_t ld = 0;  // elements between consecutive rows; 0 = contiguous rows (ld == d)
    int groups = 1;  // block-diagonal form: channel groups of d side by side in a row
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

// Column-sharded (tensor-parallel) call: the g blocks and the sign rule.
struct TpCall {
    wht::TpParts xs;    // the g blocks of x (this rank's own and the peers')
    wht::TpParts dys;   // backward only
    wht::TpParts as;    // backward only: every rank's a block
    int g;
    int r;
    unsigned neg_mask;  // bit s set: H_g[s][r] = -1
    float scale;        // 1/sqrt(g*w)
};

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

// One persistent CTA per SM (tcgen05 family): the kernel's shared-memory need alone keeps a second
// CTA off the SM, which the kernel relies on when it allocates tensor memory.
template <typename Kernel>
int prepare_umma(Kernel kernel, int smem, int dev, int* cache) {
    if (cache[dev]) return WHT_OK;
    WHT_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cache[dev] = 1;
    return WHT_OK;
}

// ---- family_misc.cu: second pass of the backward, gradient sums, copy yardstick
// da = scale * (sum of the partials' first slots), db = sum of their second slots; `groups` channel groups
// of d channels each (block-diagonal form), group k's partials, da and db following those of group k - 1
int launch_finalize(const float* parts, int nparts, int d, float scale, float* da, float* db, cudaStream_t s,
                    int groups = 1);
int launch_copy_rows(const void* src, void* dst, long long n16, int sms, cudaStream_t s);

// Common tail of every backward launcher: size the scratch, check it, launch, then the second pass
// (`grid` is the CTA count per channel group).
template <typename Launch>
int run_bwd_with_grid(const BwdArgs& g, const Ctx& c, int grid, int d, Launch launch, float scale = 0.0f) {
    *g.need = static_cast<size_t>(grid) * c.groups * 2 * d * sizeof(float);
    if (g.query_only) return WHT_OK;
    if (*g.need > 0 && (g.ws == nullptr || g.ws_bytes < *g.need)) return WHT_ERR_WORKSPACE;
    if (grid > 0) {
        launch(grid);
        WHT_CUDA_TRY(cudaGetLastError());
    }
    return launch_finalize(static_cast<const float*>(g.ws), grid, d, scale > 0.0f ? scale : inv_sqrt(d), g.da, g.db,
                           c.stream, c.groups);
}

// ---- one dispatch function per family and direction (dtype: a wht_dtype; log2 of the width)
int bfly_fwd(int logd, int dtype, const FwdArgs& f, const Ctx& c);                      // family_bfly_fwd.cu
int bfly_bwd(int logd, int dtype, const BwdArgs& g, const Ctx& c);                      // family_bfly_bwd.cu
int bfly_fwd_tp(int logw, int dtype, const TpCall& t, const FwdArgs& f, const Ctx& c);  // family_tp.cu
int bfly_bwd_tp(int logw, int dtype, const TpCall& t, const BwdArgs& g, const Ctx& c);
int mma_fwd(int logd, int dtype, bool few_rows, bool streamed, const FwdArgs& f, const Ctx& c);  // family_mma.cu
int mma_bwd(int logd, int dtype, bool streamed, const BwdArgs& g, const Ctx& c);
int umma_fwd(int logd, int dtype, const FwdArgs& f, const Ctx& c);                      // family_umma_fwd.cu
int umma_fwd_tp(int logw, int dtype, const TpCall& t, const FwdArgs& f, const Ctx& c);
// g_hi_lo: g enters the second product as a bf16 pair hi + lo (default) or rounded to bf16 once
// half_size: products with H_64 instead of H_128 (d <= 4096; wider rows take the full-size kernel)
int umma_bwd(int logd, int dtype, bool g_hi_lo, bool half_size, const BwdArgs& g, const Ctx& c);  // family_umma_bwd.cu

// Self-test of the bounded waits (family_umma_fwd.cu): a one-CTA kernel whose wait runs out after limit_us.
int launch_wait_expiry_selftest(uint32_t limit_us, unsigned int* out, cudaStream_t s);

// g >= 2 ranks, bf16 rows, 1024 <= w <= 4096                                          // family_umma_tp.cu
int umma_bwd_tp(int logw, int dtype, bool g_hi_lo, const TpCall& t, const BwdArgs& g, const Ctx& c);

// The kernels that wait with a bound record an expired wait in a device word of their own translation
// unit; each of these reads that word, clears it, and reports whether it was set.
int take_device_error_mma(unsigned* flag);
int take_device_error_umma_fwd(unsigned* flag);
int take_device_error_umma_bwd(unsigned* flag);
int take_device_error_umma_tp(unsigned* flag);

// Defines one of the three readers above in the translation unit that includes the waiting kernels.
#define WHT_DEFINE_DEVICE_ERROR_READER(name)                                                         \
    int name(unsigned* flag) {                                                                       \
        unsigned v = 0;                                                                              \
        WHT_CUDA_TRY(cudaMemcpyFromSymbol(&v, ::wht::g_wht_device_error, sizeof(v)));                \
        if (v != 0) {                                                                                \
            const unsigned zero = 0;                                                                 \
            WHT_CUDA_TRY(cudaMemcpyToSymbol(::wht::g_wht_device_error, &zero, sizeof(zero)));        \
        }                                                                                            \
        *flag = v;                                                                                   \
        return WHT_OK;                                                                               \
    }

}  // namespace wht_host
