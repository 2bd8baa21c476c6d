// Butterfly family, backward: instantiations and launch geometry.
#include "bfly_kernels.cuh"
#include "host_common.h"

namespace wht_host {

using namespace wht;

namespace {

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

template <typename TIO, typename TP>
int dispatch(int logd, const BwdArgs& g, const Ctx& c) {
    switch (logd) {
#define M(L) case L: return launch_bfly_bwd<L, TIO, TP>(g, c);
        M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int bfly_bwd(int logd, int dtype, const BwdArgs& g, const Ctx& c) {
    switch (dtype) {
        case WHT_F32: return dispatch<float, float>(logd, g, c);
        case WHT_BF16: return dispatch<__nv_bfloat16, __nv_bfloat16>(logd, g, c);
        default: return dispatch<__nv_bfloat16, float>(logd, g, c);
    }
}

}  // namespace wht_host
