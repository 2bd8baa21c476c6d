// C ABI of the library (see include/wht_affine.h): argument checks, kernel
// selection, launch geometry and the library-owned backward scratch buffer.
#include "../../include/wht_affine.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "bfly_kernels.cuh"
#include "mma_kernels.cuh"

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
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess) return 0;
    cache[dev] = n > 0 ? n : 0;
    return cache[dev];
}

long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }

// ------------------------------------------------------------------ butterfly family
template <int LOGD, typename TIO, typename TP>
int launch_bfly_fwd(const void* x, const void* a, const void* b, void* y, int64_t T,
                    int dev, int sms, cudaStream_t s) {
    using Geo = BflyGeo<LOGD>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_fwd_kernel<LOGD, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, dev, occ);
    if (per_sm <= 0) return cuda_fail(cudaGetLastError());
    const long long tiles = ceil_div(T, Geo::R);
    const long long cap = static_cast<long long>(sms) * per_sm;
    const unsigned grid = static_cast<unsigned>(tiles < cap ? tiles : cap);
    const float rs = static_cast<float>(1.0 / sqrt(static_cast<double>(Geo::D)));
    kernel<<<grid, Geo::THREADS, Geo::SMEM_FWD, s>>>(
        static_cast<const TIO*>(x), static_cast<const TP*>(a), static_cast<const TP*>(b),
        static_cast<TIO*>(y), static_cast<long long>(T), rs);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD>
int bfly_bwd_grid(int64_t T, int sms, int per_sm) {
    using Geo = BflyGeo<LOGD>;
    const long long tiles = ceil_div(T, Geo::R);
    const long long cap = static_cast<long long>(sms) * per_sm;
    return static_cast<int>(tiles < cap ? tiles : cap);
}

template <int LOGD, typename TIO, typename TP>
int launch_bfly_bwd(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                    int64_t T, void* ws, size_t ws_bytes, bool query_only, size_t* need,
                    int dev, int sms, cudaStream_t s) {
    using Geo = BflyGeo<LOGD>;
    static int occ[kMaxDevices] = {};
    auto kernel = bfly_bwd_kernel<LOGD, TIO, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, dev, occ);
    if (per_sm <= 0) return cuda_fail(cudaGetLastError());
    const int grid = bfly_bwd_grid<LOGD>(T, sms, per_sm);
    *need = static_cast<size_t>(grid) * 2 * Geo::D * sizeof(float);
    if (query_only) return WHT_OK;
    if (*need > 0 && (ws == nullptr || ws_bytes < *need)) return WHT_ERR_WORKSPACE;
    const float rs = static_cast<float>(1.0 / sqrt(static_cast<double>(Geo::D)));
    if (grid > 0) {
        kernel<<<grid, Geo::THREADS, Geo::SMEM_BWD, s>>>(
            static_cast<const TIO*>(dy), static_cast<const TIO*>(x), static_cast<const TP*>(a),
            static_cast<TIO*>(dx), static_cast<float*>(ws), static_cast<long long>(T), rs);
        WHT_CUDA_TRY(cudaGetLastError());
    }
    dadb_finalize_kernel<<<(2 * Geo::D + 255) / 256, 256, 0, s>>>(
        static_cast<const float*>(ws), grid, Geo::D, rs, da, db);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

#define WHT_FOR_EACH_LOGD(M) \
    M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)

template <typename TIO, typename TP>
int dispatch_bfly_fwd(int logd, const void* x, const void* a, const void* b, void* y, int64_t T,
                      int dev, int sms, cudaStream_t s) {
    switch (logd) {
#define M(L) case L: return launch_bfly_fwd<L, TIO, TP>(x, a, b, y, T, dev, sms, s);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TIO, typename TP>
int dispatch_bfly_bwd(int logd, const void* dy, const void* x, const void* a, void* dx, float* da,
                      float* db, int64_t T, void* ws, size_t ws_bytes, bool query_only, size_t* need,
                      int dev, int sms, cudaStream_t s) {
    switch (logd) {
#define M(L) case L: return launch_bfly_bwd<L, TIO, TP>(dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s);
        WHT_FOR_EACH_LOGD(M)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}


// ------------------------------------------------------------------ tensor-core family
template <int LOGD, int TB, int RG, typename TP>
int launch_mma_fwd(const void* x, const void* a, const void* b, void* y, int64_t T,
                   int dev, int sms, cudaStream_t s) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_fwd_kernel<LOGD, TB, RG, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, dev, occ);
    if (per_sm <= 0) return cuda_fail(cudaGetLastError());
    const long long tiles = ceil_div(T, RG);
    const long long cap = static_cast<long long>(sms) * per_sm;
    const unsigned grid = static_cast<unsigned>(tiles < cap ? tiles : cap);
    const float rs = static_cast<float>(1.0 / sqrt(static_cast<double>(Geo::D)));
    kernel<<<grid, Geo::THREADS, Geo::SMEM_FWD, s>>>(
        static_cast<const __nv_bfloat16*>(x), static_cast<const TP*>(a), static_cast<const TP*>(b),
        static_cast<__nv_bfloat16*>(y), static_cast<long long>(T), rs);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int TB, int RG, typename TP>
int launch_mma_bwd(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                   int64_t T, void* ws, size_t ws_bytes, bool query_only, size_t* need,
                   int dev, int sms, cudaStream_t s) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_bwd_kernel<LOGD, TB, RG, TP>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, dev, occ);
    if (per_sm <= 0) return cuda_fail(cudaGetLastError());
    const long long tiles = ceil_div(T, RG);
    const long long cap = static_cast<long long>(sms) * per_sm;
    const int grid = static_cast<int>(tiles < cap ? tiles : cap);
    *need = static_cast<size_t>(grid) * 2 * Geo::D * sizeof(float);
    if (query_only) return WHT_OK;
    if (*need > 0 && (ws == nullptr || ws_bytes < *need)) return WHT_ERR_WORKSPACE;
    const float rs = static_cast<float>(1.0 / sqrt(static_cast<double>(Geo::D)));
    if (grid > 0) {
        kernel<<<grid, Geo::THREADS, Geo::SMEM_BWD, s>>>(
            static_cast<const __nv_bfloat16*>(dy), static_cast<const __nv_bfloat16*>(x),
            static_cast<const TP*>(a), static_cast<__nv_bfloat16*>(dx), static_cast<float*>(ws),
            static_cast<long long>(T), rs);
        WHT_CUDA_TRY(cudaGetLastError());
    }
    dadb_finalize_kernel<<<(2 * Geo::D + 255) / 256, 256, 0, s>>>(
        static_cast<const float*>(ws), grid, Geo::D, rs, da, db);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

// Row splits (LOGD, TB, RG) of the tensor-core family.  `wide` spreads a row over
// more warps (lower latency per row, used for decode and as tuning alternative).
template <typename TP>
int dispatch_mma_fwd(int logd, bool wide, const void* x, const void* a, const void* b, void* y,
                     int64_t T, int dev, int sms, cudaStream_t s) {
    switch (logd) {
        case 9: return launch_mma_fwd<9, 1, 4, TP>(x, a, b, y, T, dev, sms, s);
        case 10: return wide ? launch_mma_fwd<10, 1, 2, TP>(x, a, b, y, T, dev, sms, s)
                             : launch_mma_fwd<10, 2, 4, TP>(x, a, b, y, T, dev, sms, s);
        case 11: return wide ? launch_mma_fwd<11, 2, 2, TP>(x, a, b, y, T, dev, sms, s)
                             : launch_mma_fwd<11, 3, 4, TP>(x, a, b, y, T, dev, sms, s);
        case 12: return wide ? launch_mma_fwd<12, 2, 1, TP>(x, a, b, y, T, dev, sms, s)
                             : launch_mma_fwd<12, 3, 2, TP>(x, a, b, y, T, dev, sms, s);
        case 13: return launch_mma_fwd<13, 3, 1, TP>(x, a, b, y, T, dev, sms, s);
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TP>
int dispatch_mma_bwd(int logd, bool wide, const void* dy, const void* x, const void* a, void* dx,
                     float* da, float* db, int64_t T, void* ws, size_t ws_bytes, bool query_only,
                     size_t* need, int dev, int sms, cudaStream_t s) {
#define WHT_BWD_ARGS dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s
    switch (logd) {
        case 9: return launch_mma_bwd<9, 1, 8, TP>(WHT_BWD_ARGS);
        case 10: return wide ? launch_mma_bwd<10, 1, 4, TP>(WHT_BWD_ARGS) : launch_mma_bwd<10, 2, 8, TP>(WHT_BWD_ARGS);
        case 11: return wide ? launch_mma_bwd<11, 2, 4, TP>(WHT_BWD_ARGS) : launch_mma_bwd<11, 3, 4, TP>(WHT_BWD_ARGS);
        case 12: return wide ? launch_mma_bwd<12, 2, 2, TP>(WHT_BWD_ARGS) : launch_mma_bwd<12, 3, 2, TP>(WHT_BWD_ARGS);
        case 13: return launch_mma_bwd<13, 3, 1, TP>(WHT_BWD_ARGS);
    }
#undef WHT_BWD_ARGS
    return WHT_ERR_BAD_DIM;
}

bool mma_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 9 && logd <= 13; }

// ------------------------------------------------------------------ selection
int run_fwd(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d, int dtype,
            cudaStream_t s, bool decode) {
    int dev = 0, sms = 0;
    int rc = current_device(&dev, &sms);
    if (rc != WHT_OK) return rc;
    const int logd = log2_of(d);
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        const bool wide = decode || g_variant == 3;
        return dtype == WHT_BF16
                   ? dispatch_mma_fwd<__nv_bfloat16>(logd, wide, x, a, b, y, T, dev, sms, s)
                   : dispatch_mma_fwd<float>(logd, wide, x, a, b, y, T, dev, sms, s);
    }
    switch (dtype) {
        case WHT_F32: return dispatch_bfly_fwd<float, float>(logd, x, a, b, y, T, dev, sms, s);
        case WHT_BF16: return dispatch_bfly_fwd<__nv_bfloat16, __nv_bfloat16>(logd, x, a, b, y, T, dev, sms, s);
        default: return dispatch_bfly_fwd<__nv_bfloat16, float>(logd, x, a, b, y, T, dev, sms, s);
    }
}

int run_bwd(const void* dy, const void* x, const void* a, void* dx, float* da, float* db, int64_t T,
            int32_t d, int dtype, void* ws, size_t ws_bytes, bool query_only, size_t* need,
            cudaStream_t s) {
    int dev = 0, sms = 0;
    int rc = current_device(&dev, &sms);
    if (rc != WHT_OK) return rc;
    const int logd = log2_of(d);
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        const bool wide = g_variant != 3;
        return dtype == WHT_BF16
                   ? dispatch_mma_bwd<__nv_bfloat16>(logd, wide, dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s)
                   : dispatch_mma_bwd<float>(logd, wide, dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s);
    }
    switch (dtype) {
        case WHT_F32:
            return dispatch_bfly_bwd<float, float>(logd, dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s);
        case WHT_BF16:
            return dispatch_bfly_bwd<__nv_bfloat16, __nv_bfloat16>(logd, dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s);
        default:
            return dispatch_bfly_bwd<__nv_bfloat16, float>(logd, dy, x, a, dx, da, db, T, ws, ws_bytes, query_only, need, dev, sms, s);
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

}  // namespace

extern "C" {

int wht_affine_fwd(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d,
                   int dtype, void* stream) {
    int rc = check_fwd_args(x, a, b, y, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (T == 0) return WHT_OK;
    return run_fwd(x, a, b, y, T, d, dtype, static_cast<cudaStream_t>(stream), false);
}

int wht_affine_fwd_decode(const void* x, const void* a, const void* b, void* y, int64_t T, int32_t d,
                          int dtype, void* stream) {
    int rc = check_fwd_args(x, a, b, y, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (T == 0) return WHT_OK;
    return run_fwd(x, a, b, y, T, d, dtype, static_cast<cudaStream_t>(stream), true);
}

size_t wht_affine_bwd_workspace_bytes(int64_t T, int32_t d, int dtype) {
    if (check_common(T, d, dtype) != WHT_OK) return 0;
    size_t need = 0;
    if (run_bwd(nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, T, d, dtype, nullptr, 0, true,
                &need, nullptr) != WHT_OK)
        return 0;
    return need;
}

int wht_affine_bwd_ws(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                      int64_t T, int32_t d, int dtype, void* workspace, size_t workspace_bytes,
                      void* stream) {
    int rc = check_bwd_args(dy, x, a, dx, da, db, T, d, dtype);
    if (rc != WHT_OK) return rc;
    if (workspace && !aligned16(workspace)) return WHT_ERR_MISALIGNED;
    size_t need = 0;
    return run_bwd(dy, x, a, dx, da, db, T, d, dtype, workspace, workspace_bytes, false, &need,
                   static_cast<cudaStream_t>(stream));
}

int wht_affine_bwd(const void* dy, const void* x, const void* a, void* dx, float* da, float* db,
                   int64_t T, int32_t d, int dtype, void* stream) {
    int rc = check_bwd_args(dy, x, a, dx, da, db, T, d, dtype);
    if (rc != WHT_OK) return rc;
    size_t need = 0;
    rc = run_bwd(nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, T, d, dtype, nullptr, 0, true,
                 &need, nullptr);
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
    return run_bwd(dy, x, a, dx, da, db, T, d, dtype, ws, ws_bytes, false, &need,
                   static_cast<cudaStream_t>(stream));
}

int wht_affine_set_variant(int variant) {
    if (variant < 0 || variant > 3) return WHT_ERR_BAD_VARIANT;
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
    const long long want = ceil_div(n16, 256);
    const long long cap = static_cast<long long>(sms) * 8;
    copy_rows_kernel<<<static_cast<unsigned>(want < cap ? want : cap), 256, 0,
                       static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), n16);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
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
