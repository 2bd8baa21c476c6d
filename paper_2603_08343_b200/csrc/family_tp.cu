// Column-sharded (tensor-parallel) form on the butterfly kernels: instantiations and launch geometry.
#include "host_common.h"
#include "tp_kernels.cuh"

namespace wht_host {

using namespace wht;

namespace {

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

template <typename TIO, typename TP>
int dispatch_fwd(int logw, const TpCall& t, const FwdArgs& f, const Ctx& c) {
    switch (logw) {
#define M(L) case L: return launch_bfly_fwd_tp<L, TIO, TP>(t, f, c);
        M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

template <typename TIO, typename TP>
int dispatch_bwd(int logw, const TpCall& t, const BwdArgs& g, const Ctx& c) {
    switch (logw) {
#define M(L) case L: return launch_bfly_bwd_tp<L, TIO, TP>(t, g, c);
        M(3) M(4) M(5) M(6) M(7) M(8) M(9) M(10) M(11) M(12) M(13) M(14) M(15)
#undef M
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int bfly_fwd_tp(int logw, int dtype, const TpCall& t, const FwdArgs& f, const Ctx& c) {
    switch (dtype) {
        case WHT_F32: return dispatch_fwd<float, float>(logw, t, f, c);
        case WHT_BF16: return dispatch_fwd<__nv_bfloat16, __nv_bfloat16>(logw, t, f, c);
        default: return dispatch_fwd<__nv_bfloat16, float>(logw, t, f, c);
    }
}

int bfly_bwd_tp(int logw, int dtype, const TpCall& t, const BwdArgs& g, const Ctx& c) {
    switch (dtype) {
        case WHT_F32: return dispatch_bwd<float, float>(logw, t, g, c);
        case WHT_BF16: return dispatch_bwd<__nv_bfloat16, __nv_bfloat16>(logw, t, g, c);
        default: return dispatch_bwd<__nv_bfloat16, float>(logw, t, g, c);
    }
}

}  // namespace wht_host
