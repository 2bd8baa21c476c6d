// tcgen05 family, forward (plain, fused residual, column-sharded): instantiations and launch geometry.
#include "host_common.h"
#include "umma_kernels.cuh"

namespace wht_host {

using namespace wht;

namespace {

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

// Lean form (see UmmaFwdSmem): two CTAs fit on an SM, so the next launch in the stream sets itself up while this
// one still runs.  One CTA per SM is launched all the same.
template <int LOGD, int NCOL, int STAGES, typename TP>
int launch_umma_fwd_lean(const FwdArgs& f, const Ctx& c) {
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaFwdSmem<LOGD, NCOL, STAGES, TP, false, true>;
    static_assert(2 * (L::BYTES + 1024) <= 227 * 1024 && L::TMEM_COLS == 256, "two CTAs must fit on an SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_fwd_kernel<LOGD, NCOL, STAGES, TP, false, false, true>;
    int rc = prepare_umma(kernel, L::BYTES, c.dev, ready);
    if (rc != WHT_OK) return rc;
    const int grid = capped_grid(ceil_div(c.T, Geo::ROWS), c.sms, 1);
    launch_overlapped(kernel, grid, Geo::THREADS, L::BYTES, c.stream,
                      static_cast<const __nv_bfloat16*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const __nv_bfloat16*>(nullptr), static_cast<__nv_bfloat16*>(f.y),
                      static_cast<long long>(c.T), inv_sqrt(Geo::D), TpParts{}, 1, 0u);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int NCOL, int STAGES, typename TP>
int launch_umma_fwd(const FwdArgs& f, const Ctx& c) {
    return f.resid ? launch_umma_fwd_impl<LOGD, NCOL, STAGES, TP, true>(f, c)
                   : launch_umma_fwd_impl<LOGD, NCOL, STAGES, TP, false>(f, c);
}

template <typename TP>
int dispatch_umma_fwd(int logd, const FwdArgs& f, const Ctx& c) {
    // From a dozen tiles per CTA on (and without a fused residual) the lean form: measured 2-6 % faster in long
    // runs at every width (d = 8192: 93.5 -> 87.7 us for 256 MiB of rows) and 1-2 % in bursts; with fewer tiles
    // (the Prefill config has 7 per CTA) its shorter ring and single accumulator lose (12.5 against 12.1 us).
    const long long tiles_per_cta = ceil_div(ceil_div(c.T * (1ll << logd) * 2, 32768), c.sms);
    if (!f.resid && tiles_per_cta >= 12) {
        switch (logd) {
            case 10: return launch_umma_fwd_lean<10, 128, 3, TP>(f, c);
            case 11: return launch_umma_fwd_lean<11, 128, 3, TP>(f, c);
            case 12: return launch_umma_fwd_lean<12, 128, 3, TP>(f, c);
            case 13: return launch_umma_fwd_lean<13, 128, 3, TP>(f, c);
        }
    }
    switch (logd) {
        case 10: return launch_umma_fwd<10, 128, 4, TP>(f, c);
        case 11: return launch_umma_fwd<11, 128, 4, TP>(f, c);
        case 12: return launch_umma_fwd<12, 128, 4, TP>(f, c);
        case 13: return launch_umma_fwd<13, 128, 4, TP>(f, c);
    }
    return WHT_ERR_BAD_DIM;
}

// column-sharded forward: one product per source block into one accumulator
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

}  // namespace

int umma_fwd(int logd, int dtype, const FwdArgs& f, const Ctx& c) {
    return dtype == WHT_BF16 ? dispatch_umma_fwd<__nv_bfloat16>(logd, f, c) : dispatch_umma_fwd<float>(logd, f, c);
}

int umma_fwd_tp(int logw, int dtype, const TpCall& t, const FwdArgs& f, const Ctx& c) {
    return dtype == WHT_BF16 ? dispatch_umma_fwd_tp<__nv_bfloat16>(logw, t, f, c)
                             : dispatch_umma_fwd_tp<float>(logw, t, f, c);
}

int launch_wait_expiry_selftest(uint32_t limit_us, unsigned int* out, cudaStream_t s) {
    // limit_us of waiting in all: parked try_waits of up to 20 us each, then polls 256 ns apart
    const uint32_t park = limit_us / 20u + 1u;
    const uint32_t spin = limit_us * 4u + 1u;
    wait_expiry_selftest_kernel<0><<<1, 64, 0, s>>>(park, spin, out);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

WHT_DEFINE_DEVICE_ERROR_READER(take_device_error_umma_fwd)

}  // namespace wht_host
