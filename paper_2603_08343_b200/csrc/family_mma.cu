// mma.sync family (direct row loads and streamed rows): instantiations and launch geometry.
#include "host_common.h"
#include "mma_pipe_kernels.cuh"

namespace wht_host {

using namespace wht;

namespace {

// CTAs along x: enough to fill the device, shared out over the channel groups of the block-diagonal form
int grid_x(const Ctx& c, int rows_per_cta, int per_sm) {
    const int grid = capped_grid(ceil_div(c.T, rows_per_cta), c.sms, per_sm);
    return c.groups > 1 ? (grid / c.groups > 0 ? grid / c.groups : 1) : grid;
}

template <int LOGD, int TB, int RG, typename TP, typename TIO = __nv_bfloat16>
int launch_mma_fwd(const FwdArgs& f, const Ctx& c) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_fwd_kernel<LOGD, TB, RG, TP, TIO>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_FWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = grid_x(c, RG, per_sm);
    launch_overlapped(kernel, dim3(grid, c.groups), Geo::THREADS, Geo::SMEM_FWD, c.stream,
                      static_cast<const TIO*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
                      static_cast<const TIO*>(f.resid), static_cast<TIO*>(f.y),
                      static_cast<long long>(c.T), static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int TB, int RG, typename TP, typename TIO = __nv_bfloat16>
int launch_mma_bwd(const BwdArgs& g, const Ctx& c) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_bwd_kernel<LOGD, TB, RG, TP, TIO>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM_BWD, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    int grid = grid_x(c, RG, per_sm);
    // every CTA publishes 2 d partial sums: keep them within 16 MiB (the scratch promised to suffice for
    // d <= 8192) where that still leaves a CTA per SM
    const int cap = static_cast<int>((16u << 20) / (2u * Geo::D * sizeof(float) * c.groups));
    if (cap >= c.sms && grid > cap) grid = cap;
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        kernel<<<dim3(n, c.groups), Geo::THREADS, Geo::SMEM_BWD, c.stream>>>(
            static_cast<const TIO*>(g.dy), static_cast<const TIO*>(g.x),
            static_cast<const TP*>(g.a), static_cast<TIO*>(g.dx), static_cast<float*>(g.ws),
            static_cast<long long>(c.T), static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    });
}

template <int LOGD, int TB, int RG, int S, int MINB, typename TP, typename TIO = __nv_bfloat16>
int launch_mma_fwd_pipe(const FwdArgs& f, const Ctx& c) {
    using Geo = PipeGeo<LOGD, TB, RG, S, false, sizeof(TIO)>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_fwd_pipe_kernel<LOGD, TB, RG, S, MINB, TP, TIO>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = grid_x(c, RG, per_sm);
    kernel<<<dim3(grid, c.groups), Geo::THREADS, Geo::SMEM, c.stream>>>(
        static_cast<const TIO*>(f.x), static_cast<const TP*>(f.a), static_cast<const TP*>(f.b),
        static_cast<const TIO*>(f.resid), static_cast<TIO*>(f.y), static_cast<long long>(c.T),
        static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

template <int LOGD, int TB, int RG, int S, int MINB, typename TP, typename TIO = __nv_bfloat16>
int launch_mma_bwd_pipe(const BwdArgs& g, const Ctx& c) {
    using Geo = PipeGeo<LOGD, TB, RG, S, true, sizeof(TIO)>;
    static int occ[kMaxDevices] = {};
    auto kernel = mma_bwd_pipe_kernel<LOGD, TB, RG, S, MINB, TP, TIO>;
    const int per_sm = resident_ctas(kernel, Geo::THREADS, Geo::SMEM, c.dev, occ);
    if (per_sm <= 0) return occupancy_fail();
    const int grid = grid_x(c, RG, per_sm);
    return run_bwd_with_grid(g, c, grid, Geo::D, [&](int n) {
        kernel<<<dim3(n, c.groups), Geo::THREADS, Geo::SMEM, c.stream>>>(
            static_cast<const TIO*>(g.dy), static_cast<const TIO*>(g.x),
            static_cast<const TP*>(g.a), static_cast<TIO*>(g.dx), static_cast<float*>(g.ws),
            static_cast<long long>(c.T), static_cast<long long>(c.ld ? c.ld : Geo::D), inv_sqrt(Geo::D));
    });
}

// How a row is split for each d: (TB = log2 chunks per thread, RG = rows in flight
// per CTA, S = ring depth).  `few_rows` picks the direct-load kernels with a row
// spread over more warps (lowest latency per row: decode and small batches).
template <typename TP>
int dispatch_mma_fwd(int logd, bool few_rows, bool streamed, const FwdArgs& f, const Ctx& c) {
    if (few_rows) {
        switch (logd) {
            case 8: return launch_mma_fwd<8, 0, 8, TP>(f, c);
            case 9: return launch_mma_fwd<9, 1, 4, TP>(f, c);
            case 10: return launch_mma_fwd<10, 1, 2, TP>(f, c);
            case 11: return launch_mma_fwd<11, 2, 2, TP>(f, c);
            // one row per CTA while every row gets an SM of its own, two beyond that
            case 12: return c.T > c.sms ? launch_mma_fwd<12, 2, 2, TP>(f, c) : launch_mma_fwd<12, 2, 1, TP>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, TP>(f, c);
        }
    } else if (!streamed) {
        switch (logd) {
            case 8: return launch_mma_fwd<8, 0, 8, TP>(f, c);
            case 9: return launch_mma_fwd<9, 1, 4, TP>(f, c);
            case 10: return launch_mma_fwd<10, 2, 4, TP>(f, c);
            case 11: return launch_mma_fwd<11, 3, 4, TP>(f, c);
            case 12: return launch_mma_fwd<12, 3, 2, TP>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, TP>(f, c);
        }
    } else {
        switch (logd) {
            case 8: return launch_mma_fwd_pipe<8, 0, 8, 4, 4, TP>(f, c);
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
            case 8: return launch_mma_bwd<8, 0, 8, TP>(g, c);
            case 9: return launch_mma_bwd<9, 1, 8, TP>(g, c);
            case 10: return launch_mma_bwd<10, 2, 8, TP>(g, c);
            case 11: return launch_mma_bwd<11, 2, 4, TP>(g, c);
            case 12: return launch_mma_bwd<12, 2, 2, TP>(g, c);
            case 13: return launch_mma_bwd<13, 3, 1, TP>(g, c);
        }
    } else {
        switch (logd) {
            case 8: return launch_mma_bwd_pipe<8, 0, 8, 4, 3, TP>(g, c);
            case 9: return launch_mma_bwd_pipe<9, 1, 16, 3, 1, TP>(g, c);
            case 10: return launch_mma_bwd_pipe<10, 2, 8, 3, 2, TP>(g, c);
            case 11: return launch_mma_bwd_pipe<11, 2, 4, 2, 2, TP>(g, c);
            case 12: return launch_mma_bwd_pipe<12, 2, 2, 2, 1, TP>(g, c);
            case 13: return launch_mma_bwd_pipe<13, 3, 1, 2, 1, TP>(g, c);
        }
    }
    return WHT_ERR_BAD_DIM;
}

// fp32 rows (fp32 parameters): every pass on three bf16 terms per operand.  A streamed row takes 4 d bytes of
// the ring (8 d in the backward), so the wide rows trade ring depth for row groups: with warps this heavy in
// registers, rows in flight across groups hide more latency than a deeper ring per group (measured).
int dispatch_mma_fwd_f32(int logd, bool few_rows, bool streamed, const FwdArgs& f, const Ctx& c) {
    if (streamed) {
        switch (logd) {
            case 8: return launch_mma_fwd_pipe<8, 0, 8, 4, 3, float, float>(f, c);
            case 9: return launch_mma_fwd_pipe<9, 1, 8, 4, 2, float, float>(f, c);
            case 10: return launch_mma_fwd_pipe<10, 1, 8, 3, 1, float, float>(f, c);
            case 11: return launch_mma_fwd_pipe<11, 2, 4, 4, 1, float, float>(f, c);
            case 12: return launch_mma_fwd_pipe<12, 3, 6, 1, 1, float, float>(f, c);
            case 13: return launch_mma_fwd_pipe<13, 3, 2, 1, 1, float, float>(f, c);
        }
    } else if (few_rows) {
        switch (logd) {
            case 8: return launch_mma_fwd<8, 0, 8, float, float>(f, c);
            case 9: return launch_mma_fwd<9, 1, 4, float, float>(f, c);
            case 10: return launch_mma_fwd<10, 1, 2, float, float>(f, c);
            case 11: return launch_mma_fwd<11, 2, 2, float, float>(f, c);
            case 12: return c.T > c.sms ? launch_mma_fwd<12, 2, 2, float, float>(f, c)
                                        : launch_mma_fwd<12, 2, 1, float, float>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, float, float>(f, c);
        }
    } else {
        switch (logd) {
            case 8: return launch_mma_fwd<8, 0, 8, float, float>(f, c);
            case 9: return launch_mma_fwd<9, 1, 4, float, float>(f, c);
            case 10: return launch_mma_fwd<10, 2, 4, float, float>(f, c);
            case 11: return launch_mma_fwd<11, 2, 4, float, float>(f, c);
            case 12: return launch_mma_fwd<12, 2, 2, float, float>(f, c);
            case 13: return launch_mma_fwd<13, 3, 1, float, float>(f, c);
        }
    }
    return WHT_ERR_BAD_DIM;
}

int dispatch_mma_bwd_f32(int logd, bool streamed, const BwdArgs& g, const Ctx& c) {
    if (streamed) {
        switch (logd) {
            case 8: return launch_mma_bwd_pipe<8, 0, 16, 3, 2, float, float>(g, c);
            case 9: return launch_mma_bwd_pipe<9, 1, 16, 2, 1, float, float>(g, c);
            case 10: return launch_mma_bwd_pipe<10, 2, 4, 3, 2, float, float>(g, c);
            case 11: return launch_mma_bwd_pipe<11, 2, 4, 2, 1, float, float>(g, c);
            case 12: return launch_mma_bwd_pipe<12, 2, 3, 1, 1, float, float>(g, c);
            // d = 8192: x and dy rows take 64 KiB of the ring each; one row group is all that fits, and the
            // direct-load kernel below is faster
        }
    }
    switch (logd) {
        case 8: return launch_mma_bwd<8, 0, 8, float, float>(g, c);
        case 9: return launch_mma_bwd<9, 1, 8, float, float>(g, c);
        case 10: return launch_mma_bwd<10, 1, 4, float, float>(g, c);
        case 11: return launch_mma_bwd<11, 2, 4, float, float>(g, c);
        case 12: return launch_mma_bwd<12, 2, 2, float, float>(g, c);
        case 13: return launch_mma_bwd<13, 3, 1, float, float>(g, c);
    }
    return WHT_ERR_BAD_DIM;
}

}  // namespace

int mma_fwd(int logd, int dtype, bool few_rows, bool streamed, const FwdArgs& f, const Ctx& c) {
    if (dtype == WHT_F32) return dispatch_mma_fwd_f32(logd, few_rows, streamed, f, c);
    return dtype == WHT_BF16 ? dispatch_mma_fwd<__nv_bfloat16>(logd, few_rows, streamed, f, c)
                             : dispatch_mma_fwd<float>(logd, few_rows, streamed, f, c);
}

int mma_bwd(int logd, int dtype, bool streamed, const BwdArgs& g, const Ctx& c) {
    if (dtype == WHT_F32) return dispatch_mma_bwd_f32(logd, streamed, g, c);
    return dtype == WHT_BF16 ? dispatch_mma_bwd<__nv_bfloat16>(logd, streamed, g, c)
                             : dispatch_mma_bwd<float>(logd, streamed, g, c);
}

WHT_DEFINE_DEVICE_ERROR_READER(take_device_error_mma)

}  // namespace wht_host
