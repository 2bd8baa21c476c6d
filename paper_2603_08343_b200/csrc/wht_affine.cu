// C ABI of the library (see include/wht_affine.h): argument checks, kernel selection and the
// library-owned backward scratch buffer.  The kernels are instantiated and launched by the
// family_*.cu files beside this one (one per kernel family, so that they compile in parallel).
#include <atomic>
#include <initializer_list>
#include <mutex>

#include "host_common.h"

namespace wht_host {

namespace {
thread_local int g_last_cuda_error = 0;
}

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return WHT_ERR_CUDA;
}

int occupancy_fail() {
    const cudaError_t e = cudaGetLastError();
    return cuda_fail(e != cudaSuccess ? e : cudaErrorLaunchOutOfResources);
}

}  // namespace wht_host

namespace {

using namespace wht_host;
using wht::kTpMaxRanks;
using wht::TpParts;

int g_variant = 0;
int g_bwd_operand_mode = 0;

struct DeviceState {
    int sm_count = 0;
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

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

size_t elem_bytes(int dtype) { return dtype == WHT_F32 ? 4 : 2; }

// Every allocation the library makes for itself goes through here, so that tests can make it fail.
std::atomic<int> g_fail_allocations{0};
cudaError_t library_malloc(void** p, size_t bytes) {
    int pending = g_fail_allocations.load();
    while (pending > 0 && !g_fail_allocations.compare_exchange_weak(pending, pending - 1)) {}
    if (pending > 0) {
        *p = nullptr;
        return cudaErrorMemoryAllocation;  // injected: the allocator is not called
    }
    return cudaMalloc(p, bytes);
}

#ifdef WHT_DEBUG
// Debug build (-DWHT_DEBUG): every output and scratch buffer of a compute call is replaced by a device
// buffer of the library's own with a guard region on either side, filled with a canary byte.  After the
// kernels have run the stream is synchronised, the guards are read back and compared, and only then is
// the payload copied into the caller's tensor.  A kernel that writes outside its output shows up as
// WHT_ERR_GUARD instead of as silent corruption of a neighbouring tensor.  Slow by design (allocation,
// synchronisation and a copy per call); the kernels themselves are the ones of the regular build.
constexpr size_t kGuardBytes = 4096;
constexpr unsigned char kCanary = 0xA5;

class GuardedBuffer {
  public:
    GuardedBuffer() = default;
    GuardedBuffer(const GuardedBuffer&) = delete;
    GuardedBuffer& operator=(const GuardedBuffer&) = delete;
    ~GuardedBuffer() { if (base_) cudaFree(base_); }

    int init(size_t bytes, cudaStream_t s) {
        bytes_ = bytes;
        padded_ = (bytes + 15) / 16 * 16;
        const cudaError_t err = library_malloc(&base_, padded_ + 2 * kGuardBytes);
        if (err != cudaSuccess) {
            cudaGetLastError();
            g_last_cuda_error = static_cast<int>(err);
            base_ = nullptr;
            return WHT_ERR_WORKSPACE;
        }
        WHT_CUDA_TRY(cudaMemsetAsync(base_, kCanary, kGuardBytes, s));
        WHT_CUDA_TRY(cudaMemsetAsync(static_cast<unsigned char*>(base_) + kGuardBytes + padded_, kCanary, kGuardBytes, s));
        return WHT_OK;
    }
    void* data() const { return static_cast<unsigned char*>(base_) + kGuardBytes; }

    // Waits for the stream, checks both guards, then hands the payload to `user` (none for scratch).
    int finish(void* user, cudaStream_t s) {
        WHT_CUDA_TRY(cudaStreamSynchronize(s));
        unsigned char host[2][kGuardBytes];
        WHT_CUDA_TRY(cudaMemcpy(host[0], base_, kGuardBytes, cudaMemcpyDeviceToHost));
        WHT_CUDA_TRY(cudaMemcpy(host[1], static_cast<unsigned char*>(base_) + kGuardBytes + padded_, kGuardBytes,
                                cudaMemcpyDeviceToHost));
        for (int side = 0; side < 2; ++side)
            for (size_t i = 0; i < kGuardBytes; ++i)
                if (host[side][i] != kCanary) return WHT_ERR_GUARD;
        if (user && bytes_ > 0) {
            WHT_CUDA_TRY(cudaMemcpyAsync(user, data(), bytes_, cudaMemcpyDeviceToDevice, s));
            WHT_CUDA_TRY(cudaStreamSynchronize(s));
        }
        return WHT_OK;
    }

  private:
    void* base_ = nullptr;
    size_t bytes_ = 0, padded_ = 0;
};
#endif

int check_common(int64_t T, int32_t d, int dtype) {
    if (dtype != WHT_F32 && dtype != WHT_BF16 && dtype != WHT_BF16_PF32) return WHT_ERR_BAD_DTYPE;
    if (!is_pow2(d) || d < 8 || d > 32768) return WHT_ERR_BAD_DIM;
    if (T < 0) return WHT_ERR_BAD_T;
    return WHT_OK;
}

bool umma_fwd_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 10 && logd <= 13; }
bool umma_bwd_supported(int logd, int dtype) { return dtype != WHT_F32 && logd >= 10 && logd <= 13; }

// Rows of 256 ... 8192 elements (d = 256: two chained H_16 passes on one chunk per thread), bf16 or fp32
bool mma_supported(int logd, int /*dtype*/) { return logd >= 8 && logd <= 13; }

// The persistent tcgen05 kernels win once there are a few hundred 32 KiB tiles (measured
// cross-over against the direct-load kernels, CUDA-graph replay, d = 1024 ... 8192).
bool enough_work_for_tiles(int64_t T, int32_t d) {
    const int64_t elems = T * static_cast<int64_t>(d);
    return elems >= (d >= 8192 ? (8ll << 20) : (4ll << 20));
}

// Streaming pays once every row group has several rows to pipeline.
bool enough_rows_to_stream(int64_t T, int sms) { return T >= static_cast<int64_t>(sms) * 32; }

// ------------------------------------------------------------------ selection
// `groups` > 1: block-diagonal form, d is the block width and the rows are groups * d elements apart
// (the tcgen05 kernels copy whole tiles of contiguous rows and do not apply).
int select_fwd(const FwdArgs& f, int64_t T, int32_t d, int dtype, cudaStream_t s, bool decode, int groups) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    c.groups = groups;
    if (groups > 1) c.ld = static_cast<int64_t>(groups) * d;
    const int logd = log2_of(d);
    if (groups == 1 && umma_fwd_supported(logd, dtype) &&
        (g_variant >= 4 || (g_variant == 0 && enough_work_for_tiles(T, d)))) {
        return umma_fwd(logd, dtype, f, c);
    }
    if (dtype == WHT_F32) {
        // fp32 rows: streamed tensor-core passes beat the register butterflies from d = 1024 on once there are
        // rows to pipeline (measured: d = 2048 0.73 -> 0.98 of the copy rate); below that the butterflies are at
        // 0.94 ... 0.98 already.  A forced variant >= 2 takes the mma.sync kernels at every size.
        const bool enough = !decode && enough_rows_to_stream(T, c.sms);
        if (mma_supported(logd, dtype) && (g_variant >= 2 || (g_variant == 0 && logd >= 10 && enough))) {
            const bool streamed = g_variant != 2;
            return mma_fwd(logd, dtype, /*few_rows=*/decode, streamed, f, c);
        }
        return bfly_fwd(logd, dtype, f, c);
    }
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        // rows of 256 or 512 elements: the direct-load kernels (which request a warp's next row ahead) beat
        // the streamed ones at every size (measured)
        const bool streamed = g_variant >= 3 || (g_variant == 0 && !decode && logd >= 10 && enough_rows_to_stream(T, c.sms));
        const bool few_rows = !streamed && (decode || (g_variant == 0 && T < static_cast<int64_t>(c.sms) * 4));
        return mma_fwd(logd, dtype, few_rows, streamed, f, c);
    }
    return bfly_fwd(logd, dtype, f, c);
}

int select_bwd(const BwdArgs& g, int64_t T, int32_t d, int dtype, cudaStream_t s, int groups) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    c.groups = groups;
    if (groups > 1) c.ld = static_cast<int64_t>(groups) * d;
    const int logd = log2_of(d);
    // the backward is the heavier kernel: the tcgen05 form was never slower than the others from a
    // few hundred rows on
    if (groups == 1 && umma_bwd_supported(logd, dtype) &&
        (g_variant >= 4 || (g_variant == 0 && T * static_cast<int64_t>(d) >= (1ll << 18)))) {
        // half-size products: measured 2-4 % faster in long runs at d = 1024 and 2048, 1 % slower at 4096
        const bool half_size = g_variant == 5 || (g_variant == 0 && logd <= 11);
        return umma_bwd(logd, dtype, g_bwd_operand_mode == 1, half_size, g, c);
    }
    if (dtype == WHT_F32) {
        // fp32 rows: the streamed kernels win at every width they have the shared memory for (measured: d = 256
        // 0.82 -> 0.93 of the copy rate, d = 2048 0.47 -> 0.91, d = 4096 0.37 -> 0.67).  At d = 8192 an x and a
        // dy row take 64 KiB of the ring, one row group is all that fits, and neither it nor the direct-load
        // kernel (within the 16 MiB of partial sums) beats the butterflies' 0.37.
        if (mma_supported(logd, dtype) &&
            (g_variant >= 2 || (g_variant == 0 && logd <= 12 && enough_rows_to_stream(T, c.sms)))) {
            return mma_bwd(logd, dtype, /*streamed=*/g_variant != 2, g, c);
        }
        return bfly_bwd(logd, dtype, g, c);
    }
    if (g_variant != 1 && mma_supported(logd, dtype)) {
        // d = 256: direct loads (measured); wider rows are streamed once there are enough of them
        const bool streamed = g_variant >= 3 || (g_variant == 0 && logd >= 9 && enough_rows_to_stream(T, c.sms));
        return mma_bwd(logd, dtype, streamed, g, c);
    }
    return bfly_bwd(logd, dtype, g, c);
}

// What the entry points call.  Regular build: the selection above.  Debug build: the same with every
// output (and the scratch) replaced by a guarded buffer and checked after the call.
int run_fwd(FwdArgs f, int64_t T, int32_t d, int dtype, cudaStream_t s, bool decode, int groups = 1) {
#ifdef WHT_DEBUG
    GuardedBuffer gy;
    int rc = gy.init(static_cast<size_t>(T) * groups * d * elem_bytes(dtype), s);
    if (rc != WHT_OK) return rc;
    void* const user_y = f.y;
    f.y = gy.data();
    rc = select_fwd(f, T, d, dtype, s, decode, groups);
    const int rg = gy.finish(rc == WHT_OK ? user_y : nullptr, s);
    return rc != WHT_OK ? rc : rg;
#else
    return select_fwd(f, T, d, dtype, s, decode, groups);
#endif
}

#ifdef WHT_DEBUG
// Guarded stand-ins for dx, da, db and the scratch of a backward call; `launch` runs the real selection.
template <typename Launch>
int guarded_bwd(BwdArgs g, size_t dx_bytes, size_t vec_bytes, size_t need, cudaStream_t s, Launch launch) {
    if (need > 0 && (g.ws == nullptr || g.ws_bytes < need)) return WHT_ERR_WORKSPACE;
    GuardedBuffer gdx, gda, gdb, gws;
    int rc = gdx.init(dx_bytes, s);
    if (rc == WHT_OK) rc = gda.init(vec_bytes, s);
    if (rc == WHT_OK) rc = gdb.init(vec_bytes, s);
    if (rc == WHT_OK) rc = gws.init(need, s);
    if (rc != WHT_OK) return rc;
    void* const user_dx = g.dx;
    float* const user_da = g.da;
    float* const user_db = g.db;
    g.dx = gdx.data();
    g.da = static_cast<float*>(gda.data());
    g.db = static_cast<float*>(gdb.data());
    g.ws = gws.data();
    g.ws_bytes = need;
    rc = launch(g);
    const bool ok = rc == WHT_OK;
    const int r1 = gdx.finish(ok ? user_dx : nullptr, s);
    const int r2 = gda.finish(ok ? user_da : nullptr, s);
    const int r3 = gdb.finish(ok ? user_db : nullptr, s);
    const int r4 = gws.finish(nullptr, s);
    if (!ok) return rc;
    return r1 != WHT_OK ? r1 : r2 != WHT_OK ? r2 : r3 != WHT_OK ? r3 : r4;
}
#endif

int run_bwd(const BwdArgs& g, int64_t T, int32_t d, int dtype, cudaStream_t s, int groups = 1) {
#ifdef WHT_DEBUG
    if (!g.query_only) {
        size_t need = 0;
        BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, &need};
        int rc = select_bwd(q, T, d, dtype, s, groups);
        if (rc != WHT_OK) return rc;
        *g.need = need;
        return guarded_bwd(g, static_cast<size_t>(T) * groups * d * elem_bytes(dtype),
                           static_cast<size_t>(groups) * d * sizeof(float), need, s,
                           [&](const BwdArgs& h) { return select_bwd(h, T, d, dtype, s, groups); });
    }
#endif
    return select_bwd(g, T, d, dtype, s, groups);
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

int select_bwd_tp(const TpCall& t, const BwdArgs& g, int64_t T, int32_t w, int dtype, cudaStream_t s) {
    Ctx c{T, 0, 0, s};
    int rc = current_device(&c.dev, &c.sms);
    if (rc != WHT_OK) return rc;
    const int logw = log2_of(w);
    // bf16 rows of 1024 ... 4096 channels per rank on two or more ranks: tcgen05 form (as in the plain
    // backward it pays from a few hundred rows on)
    if (dtype != WHT_F32 && logw >= 10 && logw <= 12 && t.g >= 2 &&
        (g_variant >= 4 || (g_variant == 0 && T * static_cast<int64_t>(w) >= (1ll << 18)))) {
        return umma_bwd_tp(logw, dtype, g_bwd_operand_mode == 1, t, g, c);
    }
    return bfly_bwd_tp(logw, dtype, t, g, c);
}

int run_bwd_tp(const TpCall& t, const BwdArgs& g, int64_t T, int32_t w, int dtype, cudaStream_t s) {
#ifdef WHT_DEBUG
    if (!g.query_only) {
        size_t need = 0;
        BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, &need};
        int rc = select_bwd_tp(t, q, T, w, dtype, s);
        if (rc != WHT_OK) return rc;
        *g.need = need;
        return guarded_bwd(g, static_cast<size_t>(T) * w * elem_bytes(dtype), static_cast<size_t>(w) * sizeof(float),
                           need, s, [&](const BwdArgs& h) { return select_bwd_tp(t, h, T, w, dtype, s); });
    }
#endif
    return select_bwd_tp(t, g, T, w, dtype, s);
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
            const cudaError_t err = library_malloc(&p, bytes);
            if (err != cudaSuccess) {
                cudaGetLastError();  // clear the runtime's sticky copy of an allocator failure
                g_last_cuda_error = static_cast<int>(err);
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
    return run_fwd(FwdArgs{x, a, b, y}, T, block, dtype, static_cast<cudaStream_t>(stream), false, d / block);
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
    size_t need = 0;
    const BwdArgs q{dy, x, a, dx, da, db, workspace, workspace_bytes, false, &need};
    return run_bwd(q, T, block, dtype, static_cast<cudaStream_t>(stream), d / block);
}

size_t wht_affine_bwd_grouped_workspace_bytes(int64_t T, int32_t d, int32_t block, int dtype) {
    if (check_grouped(T, d, block, dtype) != WHT_OK) return 0;
    size_t need = 0;
    BwdArgs q{nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, true, &need};
    return run_bwd(q, T, block, dtype, nullptr, d / block) == WHT_OK ? need : 0;
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
    FwdArgs f{nullptr, a, b, y};
    const int logw = log2_of(w);
    // bf16 rows of 1024 ... 4096 channels per rank with enough rows for 32 KiB tiles: tcgen05 form
    const bool tensor_core = dtype != WHT_F32 && logw >= 10 && logw <= 12 && (g_variant == 0 || g_variant >= 4) &&
                             (g_variant >= 4 || enough_work_for_tiles(T, w));
#ifdef WHT_DEBUG
    GuardedBuffer gy;
    rc = gy.init(static_cast<size_t>(T) * w * elem_bytes(dtype), c.stream);
    if (rc != WHT_OK) return rc;
    f.y = gy.data();
    rc = tensor_core ? umma_fwd_tp(logw, dtype, t, f, c) : bfly_fwd_tp(logw, dtype, t, f, c);
    const int rg = gy.finish(rc == WHT_OK ? y : nullptr, c.stream);
    return rc != WHT_OK ? rc : rg;
#else
    return tensor_core ? umma_fwd_tp(logw, dtype, t, f, c) : bfly_fwd_tp(logw, dtype, t, f, c);
#endif
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
    // the second pass of the backward with a unit scale: partial p, slot 0 = da_p, slot 1 = db_p
    return launch_finalize(parts, static_cast<int>(n), static_cast<int>(d), 1.0f, da, db,
                           static_cast<cudaStream_t>(stream));
}

int wht_affine_set_variant(int variant) {
    if (variant < 0 || variant > 5) return WHT_ERR_BAD_VARIANT;
    g_variant = variant;
    return WHT_OK;
}

int wht_affine_get_variant(void) { return g_variant; }

int wht_affine_set_bwd_operand_mode(int mode) {
    if (mode != 0 && mode != 1) return WHT_ERR_BAD_VARIANT;
    g_bwd_operand_mode = mode;
    return WHT_OK;
}

int wht_affine_get_bwd_operand_mode(void) { return g_bwd_operand_mode; }

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
    return launch_copy_rows(src, dst, n16, sms, static_cast<cudaStream_t>(stream));
}

int wht_affine_device_status(void) {
    // one status word per translation unit that holds waiting kernels: read and clear them all
    unsigned any = 0;
    for (auto take : {take_device_error_mma, take_device_error_umma_fwd, take_device_error_umma_bwd,
                      take_device_error_umma_tp}) {
        unsigned flag = 0;
        const int rc = take(&flag);
        if (rc != WHT_OK) return rc;
        any |= flag;
    }
    return any ? WHT_ERR_DEVICE_WAIT : WHT_OK;
}

int wht_affine_selftest_wait_expiry(uint32_t limit_us, unsigned int* out3, void* stream) {
    if (!out3) return WHT_ERR_NULL;
    if (limit_us == 0 || limit_us > 1000000u) return WHT_ERR_BAD_T;
    return launch_wait_expiry_selftest(limit_us, out3, static_cast<cudaStream_t>(stream));
}

int wht_affine_debug_build(void) {
#ifdef WHT_DEBUG
    return 1;
#else
    return 0;
#endif
}

int wht_affine_debug_selftest_guard(int damage) {
#ifdef WHT_DEBUG
    if (damage < 0 || damage > 2) return WHT_ERR_BAD_VARIANT;
    GuardedBuffer g;
    int rc = g.init(1000, nullptr);
    if (rc != WHT_OK) return rc;
    unsigned char* payload = static_cast<unsigned char*>(g.data());
    WHT_CUDA_TRY(cudaMemset(payload, 0, 1000));  // what a well-behaved kernel does
    // one byte just outside the payload, on either side: inside the library's own allocation
    if (damage == 1) WHT_CUDA_TRY(cudaMemset(payload - 1, 0, 1));
    if (damage == 2) WHT_CUDA_TRY(cudaMemset(payload + 1008, 0, 1));
    return g.finish(nullptr, nullptr);
#else
    (void)damage;
    return WHT_ERR_BAD_VARIANT;
#endif
}

int wht_affine_test_fail_allocations(int n) {
    if (n < 0) return WHT_ERR_BAD_VARIANT;
    return g_fail_allocations.exchange(n);
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
        case WHT_ERR_GUARD:
            return "WHT_ERR_GUARD: debug build: a kernel wrote outside an output or scratch buffer";
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
