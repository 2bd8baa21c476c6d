// Column-sharded (tensor-parallel) form: the d = g * w channels of a row are spread
// over g ranks, rank s holding the contiguous block x_s = x[:, s*w : (s+1)*w] as its
// own [T x w] tensor.  H_d = H_g (x) H_w in Sylvester order, so with the channel index
// split as (s, j') the output block of rank r is
//
//     y_r = a_r (.) ( (sum_s H_g[s][r] x_s) H_w ) / sqrt(g*w) + b_r,   H_g[s][r] = (-1)^popcount(s & r):
//
// the top log2 g stages are a signed sum of the g blocks, taken on the STORED values while
// they are loaded (from this GPU's memory for s == r, through peer mappings otherwise:
// plain 128-bit loads by each CTA for itself), and the rest is the local transform of width w.
// The exchange and the transform are one kernel: no block is written back between them.
//
// Backward of the same map for rank r:
//     z_r  = (sum_s H_g[s][r] x_s) H_w / sqrt(d)          da_r = sum_t dy_r (.) z_r,  db_r = sum_t dy_r
//     dx_r = (sum_s H_g[r][s] (a_s (.) dy_s)) H_w / sqrt(d)
// so it reads every rank's x and dy blocks (and the small a_s) and writes its own dx block.
#pragma once
#include "bfly_kernels.cuh"

namespace wht {

// Sources are fetched kTpBatch at a time: all loads of a batch are issued before the first use.
constexpr int kTpBatch = 4;

// v = sum_s sign_s * part_s[row, chunk], summed in rank order
template <typename Geo, typename TIO>
__device__ __forceinline__ void tp_load_signed_sum(const TpParts& parts, int g, unsigned neg_mask, long long row,
                                                   int t, float (&v)[Geo::C][8]) {
#pragma unroll
    for (int c = 0; c < Geo::C; ++c) {
        const long long off = row * Geo::D + (c * Geo::G + t) * 8;
#pragma unroll
        for (int e = 0; e < 8; ++e) v[c][e] = 0.0f;
#pragma unroll
        for (int s0 = 0; s0 < kTpMaxRanks; s0 += kTpBatch) {
            if (s0 < g) {
                Raw8<TIO> raw[kTpBatch];
#pragma unroll
                for (int j = 0; j < kTpBatch; ++j)
                    if (s0 + j < g) raw[j].load(static_cast<const TIO*>(parts.p[s0 + j]) + off);
#pragma unroll
                for (int j = 0; j < kTpBatch; ++j) {
                    if (s0 + j < g) {
                        float part[8];
                        raw[j].widen(part);
                        const float sgn = (neg_mask >> (s0 + j)) & 1u ? -1.0f : 1.0f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[c][e] = fmaf(part[e], sgn, v[c][e]);
                    }
                }
            }
        }
    }
}

template <int LOGW, typename TIO, typename TP>
__global__ void __launch_bounds__(BflyFwdGeo<LOGW>::THREADS)
bfly_fwd_tp_kernel(TpParts xs, int g, unsigned neg_mask, const TP* __restrict__ a, const TP* __restrict__ b, TIO* y,
                   long long T, float inv_sqrt_d) {
    using Geo = BflyFwdGeo<LOGW>;
    extern __shared__ __align__(16) float smem[];
    const int rg = threadIdx.x / Geo::G;
    const int t = threadIdx.x % Geo::G;
    float* srow = smem + (Geo::WARP_BITS > 0 ? rg * Geo::D : 0);

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
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long row = tile * Geo::R + rg;
        const bool valid = row < T;
        float v[Geo::C][8];
        if (valid) {
            tp_load_signed_sum<Geo, TIO>(xs, g, neg_mask, row, t, v);
        } else {
#pragma unroll
            for (int c = 0; c < Geo::C; ++c)
#pragma unroll
                for (int e = 0; e < 8; ++e) v[c][e] = 0.0f;
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
                store8_stream(y + row * Geo::D + (c * Geo::G + t) * 8, v[c]);
            }
        }
    }
}

// partials layout as in bfly_bwd_kernel: [gridDim.x][2][W], slot 0 without the 1/sqrt(d) factor.
template <int LOGW, typename TIO, typename TP>
__global__ void __launch_bounds__(BflyBwdGeo<LOGW>::THREADS)
bfly_bwd_tp_kernel(TpParts dys, TpParts xs, TpParts as, int g, int r, unsigned neg_mask, TIO* dx,
                   float* __restrict__ partials, long long T, float inv_sqrt_d) {
    using Geo = BflyBwdGeo<LOGW>;
    extern __shared__ __align__(16) float smem[];
    const int rg = threadIdx.x / Geo::G;
    const int t = threadIdx.x % Geo::G;
    float* srow = smem + rg * Geo::D;

    float da_acc[Geo::C][8], db_acc[Geo::C][8];
#pragma unroll
    for (int c = 0; c < Geo::C; ++c) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { da_acc[c][e] = 0.0f; db_acc[c][e] = 0.0f; }
    }

    const long long tiles = (T + Geo::R - 1) / Geo::R;
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long row = tile * Geo::R + rg;
        const bool valid = row < T;
        float v[Geo::C][8];
        if (valid) {
            tp_load_signed_sum<Geo, TIO>(xs, g, neg_mask, row, t, v);
        } else {
#pragma unroll
            for (int c = 0; c < Geo::C; ++c)
#pragma unroll
                for (int e = 0; e < 8; ++e) v[c][e] = 0.0f;
        }
        bfly_row_transform<Geo>(v, srow, t);  // v = (sum_s +-x_s) H_w, unnormalised
        // v <- sum_s +- a_s (.) dy_s; this rank's own dy block also feeds da, db
#pragma unroll
        for (int c = 0; c < Geo::C; ++c) {
            const int col = (c * Geo::G + t) * 8;
            float gsum[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) gsum[e] = 0.0f;
            if (valid) {
#pragma unroll
                for (int s0 = 0; s0 < kTpMaxRanks; s0 += kTpBatch) {
                    if (s0 < g) {
                        Raw8<TIO> raw[kTpBatch];
#pragma unroll
                        for (int j = 0; j < kTpBatch; ++j)
                            if (s0 + j < g)
                                raw[j].load(static_cast<const TIO*>(dys.p[s0 + j]) + row * Geo::D + col);
#pragma unroll
                        for (int j = 0; j < kTpBatch; ++j) {
                            const int s = s0 + j;
                            if (s < g) {
                                float part[8], av[8];
                                raw[j].widen(part);
                                load8(static_cast<const TP*>(as.p[s]) + col, av);
                                const float sgn = (neg_mask >> s) & 1u ? -1.0f : 1.0f;
#pragma unroll
                                for (int e = 0; e < 8; ++e) gsum[e] = fmaf(av[e] * sgn, part[e], gsum[e]);
                                if (s == r) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        da_acc[c][e] = fmaf(part[e], v[c][e], da_acc[c][e]);
                                        db_acc[c][e] += part[e];
                                    }
                                }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) v[c][e] = gsum[e];
        }
        if constexpr (Geo::WARP_BITS > 0) __syncthreads();  // srow is reused by the second transform
        bfly_row_transform<Geo>(v, srow, t);
        if (valid) {
#pragma unroll
            for (int c = 0; c < Geo::C; ++c) {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[c][e] *= inv_sqrt_d;
                store8_stream(dx + row * Geo::D + (c * Geo::G + t) * 8, v[c]);
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
            for (int rr = 0; rr < Geo::R; ++rr) s += smem[rr * Geo::D + j];
            out[which * Geo::D + j] = s;
        }
    }
}

}  // namespace wht
