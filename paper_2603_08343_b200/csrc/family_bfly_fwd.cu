// Butterfly family, forward: instantiations and launch geometry.
#include "bfly_kernels.cuh"
#include "host_common.h"

namespace wht_host {

using namespace wht;

namespace {

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

template <typename TIO, typename TP>
int dispatch(int logd, const FwdArgs& f, const Ctx& c) {
    switch (logd) {
#define M(L) case L: return launch_bfly_fwd<L, TIO, TP>(f, c);
        M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int bfly_fwd(int logd, int dtype, const FwdArgs& f, const Ctx& c) {
    switch (dtype) {
        case WHT_F32: return dispatch<float, float>(logd, f, c);
        case WHT_BF16: return dispatch<__nv_bfloat16, __nv_bfloat16>(logd, f, c);
        default: return dispatch<__nv_bfloat16, float>(logd, f, c);
    }
}

}  // namespace wht_host
