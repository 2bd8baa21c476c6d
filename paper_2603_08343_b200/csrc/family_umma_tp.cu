// tcgen05 family, backward of the column-sharded (tensor-parallel) form: instantiations and launch geometry.
#include "host_common.h"
#include "umma_tp_kernels.cuh"

namespace wht_host {

using namespace wht;

namespace {

template <int LOGW, typename TP, bool G_LO>
int launch_umma_bwd_tp(const TpCall& t, const BwdArgs& g, const Ctx& c) {
    constexpr int NCOL = 128, STAGES = 3;
    using Geo = UmmaGeo<LOGW, NCOL>;
    using L = UmmaBwdTpSmem<LOGW, NCOL, STAGES>;
    static_assert(L::BYTES > 116 * 1024, "must be alone on its SM");
    static int ready[kMaxDevices] = {};
    auto kernel = umma_bwd_tp_kernel<LOGW, NCOL, STAGES, TP, G_LO>;
    if (!g.query_only) {
        int rc = prepare_umma(kernel, L::BYTES, c.dev, ready);
        if (rc != WHT_OK) return rc;
    }
    const int grid = capped_grid(ceil_div(c.T, Geo::ROWS), c.sms, 1);
    return run_bwd_with_grid(
        g, c, grid, Geo::D,
        [&](int n) {
            kernel<<<n, Geo::THREADS, L::BYTES, c.stream>>>(t.dys, t.xs, t.as, t.g, t.r, t.neg_mask,
                                                            static_cast<__nv_bfloat16*>(g.dx),
                                                            static_cast<float*>(g.ws), static_cast<long long>(c.T),
                                                            t.scale);
        },
        t.scale);
}

template <typename TP, bool G_LO>
int dispatch(int logw, const TpCall& t, const BwdArgs& g, const Ctx& c) {
    switch (logw) {
        case 10: return launch_umma_bwd_tp<10, TP, G_LO>(t, g, c);
        case 11: return launch_umma_bwd_tp<11, TP, G_LO>(t, g, c);
        case 12: return launch_umma_bwd_tp<12, TP, G_LO>(t, g, c);
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int umma_bwd_tp(int logw, int dtype, bool g_hi_lo, const TpCall& t, const BwdArgs& g, const Ctx& c) {
    if (g_hi_lo)
        return dtype == WHT_BF16 ? dispatch<__nv_bfloat16, true>(logw, t, g, c) : dispatch<float, true>(logw, t, g, c);
    return dtype == WHT_BF16 ? dispatch<__nv_bfloat16, false>(logw, t, g, c) : dispatch<float, false>(logw, t, g, c);
}

WHT_DEFINE_DEVICE_ERROR_READER(take_device_error_umma_tp)

}  // namespace wht_host
