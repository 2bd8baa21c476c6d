// Streaming versions of the tensor-core assisted kernels: rows are brought into a
// shared-memory ring by the bulk async-copy engine (cp.async.bulk + mbarrier), so
// the bytes in flight per SM are set by the ring depth and not by registers or
// occupancy.  One elected lane per row group issues the copies; every wait on an
// mbarrier is bounded -- if it ever gives up, the kernel records that in
// g_wht_device_error and carries on (all barriers are still reached, copies that
// were issued are still waited for, bounded again), so a fault in the pipeline
// shows up as a status the host can read instead of a hang.
//
// Every copy is issued by one CTA for itself alone and every source is this GPU's own memory.
#pragma once
#include "mma_kernels.cuh"

namespace wht {

// set to a non-zero code by a kernel whose bounded wait expired (one word per translation unit of the
// library; the host reads and clears each of them)
static __device__ unsigned int g_wht_device_error = 0;
constexpr unsigned int kDeviceErrWaitExpired = 1;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
// 1-D bulk copy global -> this CTA's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
// The same with an L2 eviction hint: rows are read once, so their lines are marked evict-first.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void bulk_load_stream(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: about a quarter of a second of polling at the very least, far
// beyond any real copy latency.  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(64);
    }
    atomicExch(&g_wht_device_error, kDeviceErrWaitExpired);
    return false;
}

template <int LOGD, int TB, int RG, int S_, bool BWD, int ELEM_BYTES = 2>
struct PipeGeo : MmaGeo<LOGD, TB, RG> {
    using Base = MmaGeo<LOGD, TB, RG>;
    static constexpr int S = S_;                              // ring depth (rows in flight per row group)
    static constexpr int ROW_BYTES = Base::D * ELEM_BYTES;
    static constexpr int STAGE_BYTES = ROW_BYTES * (BWD ? 2 : 1);  // bwd: x row then dy row
    static constexpr int RING_BYTES = RG * S * STAGE_BYTES;
    static constexpr int XCHG_BYTES = RG * Base::XCHG_FLOATS * 4;
    static constexpr int BAR_BYTES = RG * S * 8;
    static constexpr int FOLD_BYTES = BWD ? RG * Base::D * 4 : 0;
    static constexpr int PARAM_OFFSET = imax_c(RING_BYTES + XCHG_BYTES, FOLD_BYTES);
    static constexpr int PARAM_BYTES = Base::D * 4 * (BWD ? 1 : 2);  // a/sqrt(d) [, b] as fp32
    static constexpr int BAR_OFFSET = PARAM_OFFSET + PARAM_BYTES;
    static constexpr int SMEM = BAR_OFFSET + BAR_BYTES;
};

// Per-channel vector -> shared memory as fp32 (times `scale`), in the order the
// threads read it: chunk c, half h, lane l hold elements c*256 + l*8 + h*4 .. +3 at
// float offset c*256 + h*128 + l*4, so a warp's 128-bit reads are conflict-free.
template <int D, int THREADS>
__device__ __forceinline__ void stage_params(const float* __restrict__ src, float* dst, float scale) {
    for (int i = threadIdx.x; i < D / 4; i += THREADS) {
        const float4 q = __ldg(reinterpret_cast<const float4*>(src) + i);
        const int e0 = i * 4, c = e0 >> 8, l = (e0 & 255) >> 3, h = (e0 & 7) >> 2;
        *reinterpret_cast<float4*>(dst + c * 256 + h * 128 + l * 4) =
            make_float4(q.x * scale, q.y * scale, q.z * scale, q.w * scale);
    }
}
template <int D, int THREADS>
__device__ __forceinline__ void stage_params(const __nv_bfloat16* __restrict__ src, float* dst, float scale) {
    for (int i = threadIdx.x; i < D / 4; i += THREADS) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(src) + i);
        const int e0 = i * 4, c = e0 >> 8, l = (e0 & 255) >> 3, h = (e0 & 7) >> 2;
        *reinterpret_cast<float4*>(dst + c * 256 + h * 128 + l * 4) =
            make_float4(bf16lo_to_f32(q.x) * scale, bf16hi_to_f32(q.x) * scale, bf16lo_to_f32(q.y) * scale,
                        bf16hi_to_f32(q.y) * scale);
    }
}
__device__ __forceinline__ void read_staged8(const float* base, int c, int lane, F2 (&v)[4]) {
    const float4* p = reinterpret_cast<const float4*>(base + c * 256 + lane * 4);
    const float4 q0 = p[0], q1 = p[32];
    v[0] = f2(q0.x, q0.y); v[1] = f2(q0.z, q0.w);
    v[2] = f2(q1.x, q1.y); v[3] = f2(q1.z, q1.w);
}

// ---- forward, streamed ----------------------------------------------------------
template <int LOGD, int TB, int RG, int S, int MINB, typename TP, typename TIO = __nv_bfloat16>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS, MINB)
mma_fwd_pipe_kernel(const TIO* x, const TP* __restrict__ a, const TP* __restrict__ b,
                    const TIO* resid, TIO* y, long long T, long long ld, float inv_sqrt_d) {
    using Geo = PipeGeo<LOGD, TB, RG, S, false, sizeof(TIO)>;
    using IO = MmaRowIO<TIO>;
    using Raw = typename IO::Raw;
    using X = MmaXform<Geo, IO::kStoredBf16 ? 2 : 3>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    unsigned char* ring = smem_raw + rg * (S * Geo::STAGE_BYTES);
    float* xbuf = reinterpret_cast<float*>(smem_raw + Geo::RING_BYTES) + rg * Geo::XCHG_FLOATS;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + Geo::BAR_OFFSET) + rg * S;
    const bool elected = (w == 0 && lane == 0);

    float* pa = reinterpret_cast<float*>(smem_raw + Geo::PARAM_OFFSET);
    float* pb = pa + Geo::D;
    {   // block-diagonal form: blockIdx.y picks the channel group [y*D, (y+1)*D) of rows ld wide
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        x += goff; y += goff; a += goff; b += goff;
        if (resid != nullptr) resid += goff;
    }

    if (elected) {
#pragma unroll
        for (int s = 0; s < S; ++s) mbar_init(full + s, 1);
        fence_mbar_init();
    }
    stage_params<Geo::D, Geo::THREADS>(a, pa, inv_sqrt_d);
    stage_params<Geo::D, Geo::THREADS>(b, pb, 1.0f);
    __syncthreads();

    uint32_t hf[4];
    make_h16_fragment(hf, lane);

    const long long stride = static_cast<long long>(gridDim.x) * RG;
    const long long first = static_cast<long long>(blockIdx.x) * RG + rg;
    auto issue = [&](int s, long long r) {
        mbar_expect_tx(full + s, Geo::ROW_BYTES);
        bulk_load(ring + s * Geo::STAGE_BYTES, x + r * ld, Geo::ROW_BYTES, full + s);
    };
    if (elected) {
#pragma unroll
        for (int s = 0; s < S; ++s) {
            const long long r = first + s * stride;
            if (r < T) issue(s, r);
        }
    }

    int stage = 0;
    uint32_t phase = 0;
    int parity = 0;
    for (long long row = first; row < T; row += stride) {
        mbar_wait_bounded(full + stage, phase);
        const unsigned char* st = ring + stage * Geo::STAGE_BYTES;
        Raw raw[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) raw[t] = IO::staged(st, chunk_of<Geo, false>(w, t) * 32 + lane);
        F2 m[NT][2][2];
        F2 v[NT][4];
        // pass 1 is warp-synchronous: every lane's reads of the stage are done after it
        if constexpr (IO::kStoredBf16) {
            X::pass1_raw(raw, m, hf);
        } else {
#pragma unroll
            for (int t = 0; t < NT; ++t) IO::pairs(raw[t], v[t]);
            X::pass1_f32(v, m, hf);
        }
        const long long next_row = row + S * stride;
        if constexpr (Geo::WB == 0) {
            __syncwarp();
            if (elected && next_row < T) issue(stage, next_row);
        }
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::exchange_and_top(v, xbuf + parity * Geo::XCHG_ONE, w, lane, 1 + rg);
        parity ^= 1;
        if constexpr (Geo::WB > 0) {
            // every warp of the row group has passed the exchange barrier, each after
            // its pass 1: the stage is free
            if (elected && next_row < T) issue(stage, next_row);
        }
        TIO* dst = y + row * ld;
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            F2 as[4], bs[4];
            read_staged8(pa, c, lane, as);
            read_staged8(pb, c, lane, bs);
            if (resid != nullptr) {
                const Raw r = IO::load(resid + row * ld, c * 32 + lane);
                fwd_store_chunk_res<TIO>(v[idx], as, bs, r, dst, c * 32 + lane);
            } else {
                fwd_store_chunk<TIO>(v[idx], as, bs, dst, c * 32 + lane);
            }
        }
        if (++stage == S) { stage = 0; phase ^= 1; }
    }
}

// ---- backward, streamed -----------------------------------------------------------
template <int LOGD, int TB, int RG, int S, int MINB, typename TP, typename TIO = __nv_bfloat16>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS, MINB)
mma_bwd_pipe_kernel(const TIO* dy, const TIO* x, const TP* __restrict__ a,
                    TIO* dx, float* __restrict__ partials, long long T, long long ld, float inv_sqrt_d) {
    using Geo = PipeGeo<LOGD, TB, RG, S, true, sizeof(TIO)>;
    using IO = MmaRowIO<TIO>;
    using Raw = typename IO::Raw;
    using X = MmaXform<Geo, IO::kStoredBf16 ? 2 : 3>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    unsigned char* ring = smem_raw + rg * (S * Geo::STAGE_BYTES);
    float* xbuf = reinterpret_cast<float*>(smem_raw + Geo::RING_BYTES) + rg * Geo::XCHG_FLOATS;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + Geo::BAR_OFFSET) + rg * S;
    const bool elected = (w == 0 && lane == 0);

    float* pa = reinterpret_cast<float*>(smem_raw + Geo::PARAM_OFFSET);
    {
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        dy += goff; x += goff; dx += goff; a += goff;
    }

    if (elected) {
#pragma unroll
        for (int s = 0; s < S; ++s) mbar_init(full + s, 1);
        fence_mbar_init();
    }
    stage_params<Geo::D, Geo::THREADS>(a, pa, inv_sqrt_d);
    __syncthreads();

    uint32_t hf[4];
    make_h16_fragment(hf, lane);

    F2 da_acc[NT][4], db_acc[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
#pragma unroll
        for (int j = 0; j < 4; ++j) { da_acc[t][j] = f2(0.0f, 0.0f); db_acc[t][j] = f2(0.0f, 0.0f); }
    }

    const long long stride = static_cast<long long>(gridDim.x) * RG;
    const long long first = static_cast<long long>(blockIdx.x) * RG + rg;
    auto issue = [&](int s, long long r) {
        mbar_expect_tx(full + s, Geo::STAGE_BYTES);
        bulk_load(ring + s * Geo::STAGE_BYTES, x + r * ld, Geo::ROW_BYTES, full + s);
        bulk_load(ring + s * Geo::STAGE_BYTES + Geo::ROW_BYTES, dy + r * ld, Geo::ROW_BYTES, full + s);
    };
    if (elected) {
#pragma unroll
        for (int s = 0; s < S; ++s) {
            const long long r = first + s * stride;
            if (r < T) issue(s, r);
        }
    }

    int stage = 0;
    uint32_t phase = 0;
    for (long long row = first; row < T; row += stride) {
        mbar_wait_bounded(full + stage, phase);
        const unsigned char* stx = ring + stage * Geo::STAGE_BYTES;
        const unsigned char* stdy = stx + Geo::ROW_BYTES;
        F2 m[NT][2][2];
        F2 v[NT][4];
        // u = x H, delivered in layout B
        if constexpr (IO::kStoredBf16) {
            Raw raw[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) raw[t] = IO::staged(stx, chunk_of<Geo, false>(w, t) * 32 + lane);
            X::pass1_raw(raw, m, hf);
        } else {
#pragma unroll
            for (int t = 0; t < NT; ++t) IO::pairs(IO::staged(stx, chunk_of<Geo, false>(w, t) * 32 + lane), v[t]);
            X::pass1_f32(v, m, hf);
        }
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::exchange_and_top(v, xbuf, w, lane, 1 + rg);
        // da, db partial sums and g = a (.) dy, all in layout B
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            F2 as[4];
            read_staged8(pa, c, lane, as);
            bwd_mid_chunk<TIO>(v[idx], IO::staged(stdy, c * 32 + lane), as, da_acc[idx], db_acc[idx]);
        }
        // dx = (g H)/sqrt(d): layout B in, layout A out
        X::pass1_f32(v, m, hf);  // warp-synchronous: this warp's reads of the stage are done here
        const long long next_row = row + S * stride;
        if constexpr (Geo::WB == 0) {
            __syncwarp();
            if (elected && next_row < T) issue(stage, next_row);
        }
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::exchange_and_top(v, xbuf + Geo::XCHG_ONE, w, lane, 1 + rg);
        if constexpr (Geo::WB > 0) {
            if (elected && next_row < T) issue(stage, next_row);
        }
        TIO* dst = dx + row * ld;
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) IO::store(dst, chunk_of<Geo, false>(w, idx) * 32 + lane, v[idx]);
        if (++stage == S) { stage = 0; phase ^= 1; }
    }
    bwd_publish_partials<Geo>(da_acc, db_acc, reinterpret_cast<float*>(smem_raw), partials, rg, w, lane);
}

}  // namespace wht
