// Butterfly kernel family: the FWHT of Fig. 2 on one row per thread group.
//
// Index bits of a row of d = 2^LOGD elements are split as
//     [ chunk c (log2 C) | thread t in group (log2 G) | element e (3) ]
// A thread owns C chunks of 8 contiguous elements (one 128-bit access each for
// bf16).  Stages on the e bits and the c bits run in registers, stages on the
// low 5 bits of t run across lanes with __shfl_xor_sync, and stages on the
// remaining bits of t (rows wider than one warp) run through a shared-memory
// copy of the row in radix-8 rounds.  Where the registers allow (up to 8 chunks
// in the forward, 2 in the backward, which also carries dy and the da/db
// accumulators) C is chosen so that a row stays inside ONE warp: d <= 2048 in the
// forward, d <= 512 in the backward need no shared memory and no CTA barrier.
// The 1/sqrt(d) scale, a and b are applied when the row is written out.  Works
// for every power of two 8 <= d <= 32768 and every storage type; it is also the
// only family for fp32 storage.
#pragma once
#include "wht_common.cuh"

#ifndef WHT_BFLY_FWD_MAXC
#define WHT_BFLY_FWD_MAXC 8
#endif
#ifndef WHT_BFLY_MIN_THREADS
#define WHT_BFLY_MIN_THREADS 256
#endif
#ifndef WHT_BFLY_BWD_MAXC
#define WHT_BFLY_BWD_MAXC 2
#endif

namespace wht {

template <int LOGD, int MAXC>
struct BflyGeo {
    static constexpr int D = 1 << LOGD;
    // chunks of 8 per thread: D/256 of them put the whole row in ONE warp (no shared memory, no CTA
    // barrier) -- used when MAXC (registers) allows; otherwise as few as keep the row within 1024
    // threads (measured: between those two, more chunks per thread only cost occupancy)
    static constexpr int C = (D >= 256 && D / 256 <= MAXC) ? D / 256 : imax_c(1, D / 8192);
    static constexpr int G = D / (8 * C);              // threads per row, 1..1024
    static constexpr int LOGG = ilog2_c(G);
    static constexpr int THREADS = imax_c(G, WHT_BFLY_MIN_THREADS);
    static constexpr int R = THREADS / G;              // rows per CTA tile
    static constexpr int LANE_BITS = imin_c(5, LOGG);
    static constexpr int WARP_BITS = LOGG - LANE_BITS; // stages that cross warps
    static constexpr int SMEM_ROW_BYTES = D * 4;
    static constexpr int SMEM_FWD = WARP_BITS > 0 ? R * D * 4 : 0;
    static constexpr int SMEM_BWD = R * D * 4;
    // few chunks per thread: little data in flight per thread, so the next tile's rows are
    // requested before this tile's are transformed, and a / b stay in registers
    static constexpr bool PREFETCH = C <= 2;
};
template <int LOGD> using BflyFwdGeo = BflyGeo<LOGD, WHT_BFLY_FWD_MAXC>;
template <int LOGD> using BflyBwdGeo = BflyGeo<LOGD, WHT_BFLY_BWD_MAXC>;

// One radix-2^NB round on row bits [P, P+NB) through shared memory.
template <typename Geo, int P, int NB>
__device__ __forceinline__ void bfly_smem_round(float* srow, int t) {
    constexpr int SETS = (8 * Geo::C) >> NB;
    constexpr int N = 1 << NB;
#pragma unroll
    for (int k = 0; k < SETS; ++k) {
        const int s = t + Geo::G * k;
        const int base = ((s >> P) << (P + NB)) | (s & ((1 << P) - 1));
        float r[N];
#pragma unroll
        for (int j = 0; j < N; ++j) r[j] = srow[base + (j << P)];
#pragma unroll
        for (int h = 1; h < N; h <<= 1) {
#pragma unroll
            for (int j = 0; j < N; ++j) {
                if ((j & h) == 0) {
                    const float lo = r[j], hi = r[j + h];
                    r[j] = lo + hi;
                    r[j + h] = lo - hi;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < N; ++j) srow[base + (j << P)] = r[j];
    }
}

template <typename Geo, int P, int REM>
struct BflyCrossRounds {
    static __device__ __forceinline__ void run(float* srow, int t) {
        constexpr int NB = imin_c(3, REM);
        bfly_smem_round<Geo, P, NB>(srow, t);
        __syncthreads();
        BflyCrossRounds<Geo, P + NB, REM - NB>::run(srow, t);
    }
};
template <typename Geo, int P>
struct BflyCrossRounds<Geo, P, 0> {
    static __device__ __forceinline__ void run(float*, int) {}
};

// Unnormalised H_d applied in place to the row held by one thread group.
// Every thread of the CTA must call this (it contains __syncthreads when the
// row spans several warps).
template <typename Geo>
__device__ __forceinline__ void bfly_row_transform(float (&v)[Geo::C][8], float* srow, int t) {
#pragma unroll
    for (int c = 0; c < Geo::C; ++c) bfly8(v[c]);
    // chunk bits (the top log2 C bits of the row index)
#pragma unroll
    for (int h = 1; h < Geo::C; h <<= 1) {
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            if ((c & h) == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float lo = v[c][e], hi = v[c + h][e];
                    v[c][e] = lo + hi;
                    v[c + h][e] = lo - hi;
                }
            }
        }
    }
    // lane bits: the partner's value arrives by shuffle; the upper lane of a
    // pair keeps (partner - own), the lower (own + partner)
#pragma unroll
    for (int m = 1; m < (1 << Geo::LANE_BITS); m <<= 1) {
        const float sgn = (t & m) ? -1.0f : 1.0f;
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float other = __shfl_xor_sync(kFullMask, v[c][e], m);
                v[c][e] = fmaf(v[c][e], sgn, other);
            }
        }
    }
    if constexpr (Geo::WARP_BITS > 0) {
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            float4* dst = reinterpret_cast<float4*>(srow + (c * Geo::G + t) * 8);
            dst[0] = make_float4(v[c][0], v[c][1], v[c][2], v[c][3]);
            dst[1] = make_float4(v[c][4], v[c][5], v[c][6], v[c][7]);
        }
        __syncthreads();
        BflyCrossRounds<Geo, 3 + Geo::LANE_BITS, Geo::WARP_BITS>::run(srow, t);
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            const float4* src = reinterpret_cast<const float4*>(srow + (c * Geo::G + t) * 8);
            const float4 q0 = src[0], q1 = src[1];
            v[c][0] = q0.x; v[c][1] = q0.y; v[c][2] = q0.z; v[c][3] = q0.w;
            v[c][4] = q1.x; v[c][5] = q1.y; v[c][6] = q1.z; v[c][7] = q1.w;
        }
    }
}

// 8 contiguous row elements as loaded (bf16: one 128-bit word, fp32: two), widened on use.
// Rows are touched once, so they are marked evict-first.
template <typename TIO> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
    uint4 q;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldcs(reinterpret_cast<const uint4*>(p)); }
    __device__ __forceinline__ void zero() { q = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void widen(float (&v)[8]) const {
        v[0] = bf16lo_to_f32(q.x); v[1] = bf16hi_to_f32(q.x);
        v[2] = bf16lo_to_f32(q.y); v[3] = bf16hi_to_f32(q.y);
        v[4] = bf16lo_to_f32(q.z); v[5] = bf16hi_to_f32(q.z);
        v[6] = bf16lo_to_f32(q.w); v[7] = bf16hi_to_f32(q.w);
    }
};
template <> struct Raw8<float> {
    float4 q0, q1;
    __device__ __forceinline__ void load(const float* p) {
        q0 = __ldcs(reinterpret_cast<const float4*>(p));
        q1 = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    }
    __device__ __forceinline__ void zero() { q0 = q1 = make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
    __device__ __forceinline__ void widen(float (&v)[8]) const {
        v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w;
        v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
    }
};
template <typename TIO>
__device__ __forceinline__ void load8_stream(const TIO* p, float (&v)[8]) {
    Raw8<TIO> r;
    r.load(p);
    r.widen(v);
}
__device__ __forceinline__ void store8_stream(float* p, const float (&v)[8]) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(v[4], v[5], v[6], v[7]));
}
__device__ __forceinline__ void store8_stream(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 q;
    q.x = pack_bf16x2(v[0], v[1]);
    q.y = pack_bf16x2(v[2], v[3]);
    q.z = pack_bf16x2(v[4], v[5]);
    q.w = pack_bf16x2(v[6], v[7]);
    __stcs(reinterpret_cast<uint4*>(p), q);
}

// The C chunks of one thread's share of a row, as loaded (zeros for a row past the end).
template <typename Geo, typename TIO>
__device__ __forceinline__ void bfly_load_row(const TIO* base, long long row, long long T, long long ld, int t,
                                              Raw8<TIO> (&raw)[Geo::C]) {
#pragma unroll
    for (int c = 0; c < Geo::C; ++c) {
        if (row < T) raw[c].load(base + row * ld + (c * Geo::G + t) * 8);
        else raw[c].zero();
    }
}

// ---- forward: y = a (.) (x H)/sqrt(d) + b ------------------------------------
template <int LOGD, typename TIO, typename TP>
__global__ void __launch_bounds__(BflyFwdGeo<LOGD>::THREADS)
bfly_fwd_kernel(const TIO* x, const TP* __restrict__ a, const TP* __restrict__ b, const TIO* resid, TIO* y,
                long long T, long long ld, float inv_sqrt_d) {  // ld: elements between consecutive rows (>= D)
    using Geo = BflyFwdGeo<LOGD>;
    extern __shared__ __align__(16) float smem[];
    const int rg = threadIdx.x / Geo::G;  // row group inside the CTA
    const int t = threadIdx.x % Geo::G;
    float* srow = smem + (Geo::WARP_BITS > 0 ? rg * Geo::D : 0);
    {   // block-diagonal form: blockIdx.y picks the channel group [y*D, (y+1)*D) of rows ld wide
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        x += goff; y += goff; a += goff; b += goff;
        if (resid != nullptr) resid += goff;
    }
    grid_dependency_wait();  // nothing above touched global memory
    grid_launch_dependents();

    constexpr int PC = Geo::PREFETCH ? Geo::C : 1;  // a, b in registers only when a thread has few channels
    float as[PC][8], bs[PC][8];
    if constexpr (Geo::PREFETCH) {
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            load8(a + (c * Geo::G + t) * 8, as[c]);
            load8(b + (c * Geo::G + t) * 8, bs[c]);
#pragma unroll
            for (int e = 0; e < 8; ++e) as[c][e] *= inv_sqrt_d;
        }
    }

    const long long tiles = (T + Geo::R - 1) / Geo::R;
    Raw8<TIO> raw[Geo::C];
    if constexpr (Geo::PREFETCH) {
        if (blockIdx.x < tiles) bfly_load_row<Geo, TIO>(x, blockIdx.x * static_cast<long long>(Geo::R) + rg, T, ld, t, raw);
    }
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long row = tile * Geo::R + rg;
        const bool valid = row < T;
        if constexpr (!Geo::PREFETCH) bfly_load_row<Geo, TIO>(x, row, T, ld, t, raw);
        float v[Geo::C][8];
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) raw[c].widen(v[c]);
        if constexpr (Geo::PREFETCH) {
            const long long next = tile + gridDim.x;
            if (next < tiles) bfly_load_row<Geo, TIO>(x, next * Geo::R + rg, T, ld, t, raw);
        }
        bfly_row_transform<Geo>(v, srow, t);
        if (valid) {
#pragma unroll
            for (int c = 0; c < Geo::C; ++c) {
                if constexpr (Geo::PREFETCH) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[c][e] = fmaf(v[c][e], as[c][e], bs[c][e]);
                } else {
                    float av[8], bv[8];  // L1-resident after the first tile
                    load8(a + (c * Geo::G + t) * 8, av);
                    load8(b + (c * Geo::G + t) * 8, bv);
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[c][e] = fmaf(v[c][e], av[e] * inv_sqrt_d, bv[e]);
                }
                if (resid != nullptr) {  // fused residual: summed in fp32, rounded once at the store
                    float r[8];
                    load8_stream(resid + row * ld + (c * Geo::G + t) * 8, r);
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[c][e] += r[e];
                }
                store8_stream(y + row * ld + (c * Geo::G + t) * 8, v[c]);
            }
        }
    }
}

// ---- backward: dx = ((a (.) dy) H)/sqrt(d); per-CTA partial da, db -------------
// partials layout: [gridDim.y][gridDim.x][2][D] fp32; slot 0 holds sum_t dy (.) (x H) WITHOUT
// the 1/sqrt(d) factor (the finalize pass applies it), slot 1 holds sum_t dy.
template <int LOGD, typename TIO, typename TP>
__global__ void __launch_bounds__(BflyBwdGeo<LOGD>::THREADS)
bfly_bwd_kernel(const TIO* dy, const TIO* x, const TP* __restrict__ a, TIO* dx,
                float* __restrict__ partials, long long T, long long ld, float inv_sqrt_d) {
    using Geo = BflyBwdGeo<LOGD>;
    extern __shared__ __align__(16) float smem[];
    const int rg = threadIdx.x / Geo::G;
    const int t = threadIdx.x % Geo::G;
    float* srow = smem + rg * Geo::D;
    {   // block-diagonal form: blockIdx.y picks the channel group; its partials follow the previous group's
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        dy += goff; x += goff; dx += goff; a += goff;
        partials += static_cast<size_t>(blockIdx.y) * gridDim.x * 2 * Geo::D;
    }
    grid_dependency_wait();  // nothing above touched global memory
    grid_launch_dependents();

    float da_acc[Geo::C][8], db_acc[Geo::C][8];
#pragma unroll
    for (int c = 0; c < Geo::C; ++c) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { da_acc[c][e] = 0.0f; db_acc[c][e] = 0.0f; }
    }

    const long long tiles = (T + Geo::R - 1) / Geo::R;
    Raw8<TIO> rx[Geo::C], rdy[Geo::C];
    if constexpr (Geo::PREFETCH) {
        if (blockIdx.x < tiles) {
            const long long row0 = blockIdx.x * static_cast<long long>(Geo::R) + rg;
            bfly_load_row<Geo, TIO>(x, row0, T, ld, t, rx);
            bfly_load_row<Geo, TIO>(dy, row0, T, ld, t, rdy);
        }
    }
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long row = tile * Geo::R + rg;
        const bool valid = row < T;
        if constexpr (!Geo::PREFETCH) {
            bfly_load_row<Geo, TIO>(x, row, T, ld, t, rx);
            bfly_load_row<Geo, TIO>(dy, row, T, ld, t, rdy);
        }
        float v[Geo::C][8], w[Geo::C][8];
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) { rx[c].widen(v[c]); rdy[c].widen(w[c]); }
        if constexpr (Geo::PREFETCH) {
            const long long next = tile + gridDim.x;
            if (next < tiles) {
                bfly_load_row<Geo, TIO>(x, next * Geo::R + rg, T, ld, t, rx);
                bfly_load_row<Geo, TIO>(dy, next * Geo::R + rg, T, ld, t, rdy);
            }
        }
        bfly_row_transform<Geo>(v, srow, t);  // v = x H (unnormalised)
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            float as[8];
            load8(a + (c * Geo::G + t) * 8, as);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                da_acc[c][e] = fmaf(w[c][e], v[c][e], da_acc[c][e]);
                db_acc[c][e] += w[c][e];
                v[c][e] = as[e] * w[c][e];
            }
        }
        if constexpr (Geo::WARP_BITS > 0) __syncthreads();  // srow is reused by the second transform
        bfly_row_transform<Geo>(v, srow, t);  // v = (a (.) dy) H
        if (valid) {
#pragma unroll
            for (int c = 0; c < Geo::C; ++c) {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[c][e] *= inv_sqrt_d;
                store8_stream(dx + row * ld + (c * Geo::G + t) * 8, v[c]);
            }
        }
    }

    // fold the R row groups of this CTA in a fixed order, then publish
    float* out = partials + static_cast<size_t>(blockIdx.x) * 2 * Geo::D;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        __syncthreads();
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            float4* dst = reinterpret_cast<float4*>(srow + (c * Geo::G + t) * 8);
            const float (&src)[8] = which == 0 ? da_acc[c] : db_acc[c];
            dst[0] = make_float4(src[0], src[1], src[2], src[3]);
            dst[1] = make_float4(src[4], src[5], src[6], src[7]);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < Geo::D; j += Geo::THREADS) {
            float s = 0.0f;
#pragma unroll
            for (int r = 0; r < Geo::R; ++r) s += smem[r * Geo::D + j];
            out[which * Geo::D + j] = s;
        }
    }
}

}  // namespace wht
