// tcgen05 family, backward: instantiations and launch geometry.
#include "host_common.h"
#include "umma64_kernels.cuh"

namespace wht_host {

using namespace wht;

namespace {

// H_128 in tensor memory (A_TMEM): in long runs under the power cap measured 4 % faster than the
// shared-memory operand at d = 8192 and 0-1 % at d = 2048 (less shared-memory traffic per product),
// the same in short bursts.
template <int LOGD, int NCOL, int STAGES, typename TP, bool A_TMEM, bool G_LO>
int launch_umma_bwd(const BwdArgs& g, const Ctx& c) {
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaBwdSmem<LOGD, NCOL, STAGES>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_bwd_kernel<LOGD, NCOL, STAGES, TP, A_TMEM, G_LO>;
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

// Half-size products (M = 64, d <= 4096): a quarter less energy per row in the tensor core for one more
// register stage; see umma64_kernels.cuh.
template <int LOGD, int STAGES, typename TP, bool G_LO>
int launch_umma64_bwd(const BwdArgs& g, const Ctx& c) {
    using Geo = Umma64Geo<LOGD>;
    using L = Umma64BwdSmem<LOGD, STAGES>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma64_bwd_kernel<LOGD, STAGES, TP, G_LO>;
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

template <typename TP, bool G_LO>
int dispatch_umma64_bwd(int logd, const BwdArgs& g, const Ctx& c) {
    switch (logd) {
        case 10: return launch_umma64_bwd<10, 3, TP, G_LO>(g, c);
        case 11: return launch_umma64_bwd<11, 3, TP, G_LO>(g, c);
        case 12: return launch_umma64_bwd<12, 3, TP, G_LO>(g, c);
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TP, bool G_LO>
int dispatch_umma_bwd(int logd, const BwdArgs& g, const Ctx& c) {
    switch (logd) {
        case 10: return launch_umma_bwd<10, 128, 3, TP, true, G_LO>(g, c);
        case 11: return launch_umma_bwd<11, 128, 3, TP, true, G_LO>(g, c);
        case 12: return launch_umma_bwd<12, 128, 3, TP, true, G_LO>(g, c);
        case 13: return launch_umma_bwd<13, 128, 3, TP, true, G_LO>(g, c);
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int umma_bwd(int logd, int dtype, bool g_hi_lo, bool half_size, const BwdArgs& g, const Ctx& c) {
    if (half_size && logd <= 12) {
        if (g_hi_lo)
            return dtype == WHT_BF16 ? dispatch_umma64_bwd<__nv_bfloat16, true>(logd, g, c)
                                     : dispatch_umma64_bwd<float, true>(logd, g, c);
        return dtype == WHT_BF16 ? dispatch_umma64_bwd<__nv_bfloat16, false>(logd, g, c)
                                 : dispatch_umma64_bwd<float, false>(logd, g, c);
    }
    if (g_hi_lo)
        return dtype == WHT_BF16 ? dispatch_umma_bwd<__nv_bfloat16, true>(logd, g, c)
                                 : dispatch_umma_bwd<float, true>(logd, g, c);
    return dtype == WHT_BF16 ? dispatch_umma_bwd<__nv_bfloat16, false>(logd, g, c)
                             : dispatch_umma_bwd<float, false>(logd, g, c);
}

WHT_DEFINE_DEVICE_ERROR_READER(take_device_error_umma_bwd)

}  // namespace wht_host
