// Tensor-core assisted kernel family for bf16 rows, 512 <= d <= 8192.
//
// H_d = H_2 (x) ... (x) H_2 is symmetric under any permutation of the index bits,
// so four butterfly stages on ANY four index bits are one product with H_16.  A
// warp-level mma.m16n8k16 (bf16 in, fp32 accumulate) computes D = H_16 * B for a
// 16 x 8 tile B whose 16-long columns are spread over the 4 lanes of a quad and 4
// values per thread -- i.e. it performs four stages AND the cross-lane exchange
// those stages need, which is the part that bounds the shuffle-based butterfly
// (its profile shows the shared-memory/shuffle data pipe near 80 % with DRAM
// under 30 %).
//
// Row layout.  A row of d = 2^LOGD elements is split as
//     [ warp w (WB bits) | chunk t (TB bits) | lane (5 bits) | element e (3 bits) ]
// A thread holds NT = 2^TB chunks of 8 contiguous elements, each one 128-bit load,
// at the position of its lane; lane = 4*g + q with q = index bits 3,4 and
// g = index bits 5,6,7.
//
//   pass 1  mma on bits {0, 3, 4, 1}: the bf16 pairs of a loaded 128-bit word are
//           B-fragment registers as they are (k = pair bit, q, register select).
//           Inputs are the stored bf16 values and +-1, products are exact and the
//           sum is fp32: this IS fp32 accumulation of four stages.
//   regs    fp32 butterflies on bit 2 and on chunk bits 1..TB-1.
//   pass 2  mma on bits {5, 6, 7, 8}: the accumulator fragment of pass 1 has bits
//           5,6,7 exactly where a B fragment wants k (that is the usual chaining
//           property of mma fragments); bit 8 (chunk bit 0) selects the register.
//           The fp32 operands are split into bf16 hi + lo (two mma into one
//           accumulator), which carries 16-17 significant bits into the product.
//   after pass 2 the accumulator fragment is the LOAD layout again (8 contiguous
//           elements per thread and chunk), so the row is stored with 128-bit
//           coalesced stores and no further exchange.
//   rows wider than one warp's 256*NT elements: the remaining WB bits are swapped
//           with the top WB chunk bits through shared memory (fp32, conflict-free
//           128-bit accesses, one named barrier per exchange, double-buffered),
//           then finished with fp32 butterflies in registers.
#pragma once
#include "wht_common.cuh"

namespace wht {

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                                  uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A-operand fragment of H_16 (entries +-1, exact in bf16): A[r][c] = (-1)^popcount(r & c).
__device__ __forceinline__ void make_h16_fragment(uint32_t (&a)[4], int lane) {
    const int g = lane >> 2, q = lane & 3;
    auto s = [](int r, int c) -> uint32_t { return (__popc(r & c) & 1) ? 0xBF80u : 0x3F80u; };
    a[0] = s(g, 2 * q) | (s(g, 2 * q + 1) << 16);
    a[1] = s(g + 8, 2 * q) | (s(g + 8, 2 * q + 1) << 16);
    a[2] = s(g, 2 * q + 8) | (s(g, 2 * q + 9) << 16);
    a[3] = s(g + 8, 2 * q + 8) | (s(g + 8, 2 * q + 9) << 16);
}

// fp32 pair -> bf16x2 hi (round to nearest) and bf16x2 lo (rounded remainder)
__device__ __forceinline__ void split_hi_lo(float v0, float v1, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16x2(v0, v1);
    lo = pack_bf16x2(v0 - bf16lo_to_f32(hi), v1 - bf16hi_to_f32(hi));
}

__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int LOGD, int TB, int RG_>
struct MmaGeo {
    static constexpr int D = 1 << LOGD;
    static constexpr int NT = 1 << TB;         // chunks of 8 elements per thread
    static constexpr int WB = LOGD - 8 - TB;   // stages that cross warps
    static_assert(TB >= 1 && WB >= 0 && WB <= TB, "unsupported split of the row");
    static constexpr int W = 1 << WB;          // warps per row
    static constexpr int NREST = NT / W;
    static constexpr int RG = RG_;             // rows in flight per CTA
    static constexpr int GROUP_THREADS = W * 32;
    static constexpr int THREADS = RG * GROUP_THREADS;
    static constexpr int XCHG_FLOATS = WB > 0 ? 2 * D : 0;  // per row group (double buffer)
    static constexpr int SMEM_FWD = RG * XCHG_FLOATS * 4;
    static constexpr int SMEM_BWD = imax_c(RG * XCHG_FLOATS * 4, RG * D * 4);
};

// Chunk (group of 256 elements) held in slot `idx` of a thread of warp `w`.
//   layout A: [ w | idx ]                        (what a warp loads contiguously)
//   layout B: [ idx_top | w | idx_rest ]         (after the cross-warp exchange)
template <class Geo, bool LAYOUT_B>
__device__ __forceinline__ int chunk_of(int w, int idx) {
    if constexpr (Geo::WB == 0) {
        return idx;
    } else if constexpr (!LAYOUT_B) {
        return w * Geo::NT + idx;
    } else {
        return (idx / Geo::NREST) * Geo::NT + w * Geo::NREST + (idx % Geo::NREST);
    }
}

template <class Geo>
struct MmaXform {
    static constexpr int NT = Geo::NT;

    // pass 1 on stored bf16: m[t][h][2p + r] <- bits {0,3,4,1} transformed
    static __device__ __forceinline__ void pass1_raw(const uint4 (&raw)[NT], float (&m)[NT][2][4],
                                                     const uint32_t (&hf)[4]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { m[t][0][i] = 0.0f; m[t][1][i] = 0.0f; }
            mma_bf16_m16n8k16(m[t][0], hf, raw[t].x, raw[t].y);
            mma_bf16_m16n8k16(m[t][1], hf, raw[t].z, raw[t].w);
        }
    }

    // pass 1 on fp32 values in load layout v[t][e] (hi/lo split operands)
    static __device__ __forceinline__ void pass1_f32(const float (&v)[NT][8], float (&m)[NT][2][4],
                                                     const uint32_t (&hf)[4]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t b0h, b0l, b1h, b1l;
                split_hi_lo(v[t][4 * h + 0], v[t][4 * h + 1], b0h, b0l);
                split_hi_lo(v[t][4 * h + 2], v[t][4 * h + 3], b1h, b1l);
#pragma unroll
                for (int i = 0; i < 4; ++i) m[t][h][i] = 0.0f;
                mma_bf16_m16n8k16(m[t][h], hf, b0h, b1h);
                mma_bf16_m16n8k16(m[t][h], hf, b0l, b1l);
            }
        }
    }

    // fp32 butterflies on bit 2 (h) and on chunk-slot bits 1..TB-1
    static __device__ __forceinline__ void mid_stages(float (&m)[NT][2][4]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = m[t][0][i], hi = m[t][1][i];
                m[t][0][i] = lo + hi;
                m[t][1][i] = lo - hi;
            }
        }
#pragma unroll
        for (int bit = 2; bit < NT; bit <<= 1) {
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                if ((t & bit) == 0) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float lo = m[t][h][i], hi = m[t + bit][h][i];
                            m[t][h][i] = lo + hi;
                            m[t + bit][h][i] = lo - hi;
                        }
                    }
                }
            }
        }
    }

    // pass 2 on bits {5,6,7} and chunk-slot bit 0; result v[t][e] is in load layout
    static __device__ __forceinline__ void pass2(const float (&m)[NT][2][4], float (&v)[NT][8],
                                                 const uint32_t (&hf)[4]) {
#pragma unroll
        for (int u = 0; u < NT / 2; ++u) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    uint32_t b0h, b0l, b1h, b1l;
                    split_hi_lo(m[2 * u][h][2 * p], m[2 * u][h][2 * p + 1], b0h, b0l);
                    split_hi_lo(m[2 * u + 1][h][2 * p], m[2 * u + 1][h][2 * p + 1], b1h, b1l);
                    float d[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                    mma_bf16_m16n8k16(d, hf, b0h, b1h);
                    mma_bf16_m16n8k16(d, hf, b0l, b1l);
                    v[2 * u][4 * h + 2 * p + 0] = d[0];
                    v[2 * u][4 * h + 2 * p + 1] = d[1];
                    v[2 * u + 1][4 * h + 2 * p + 0] = d[2];
                    v[2 * u + 1][4 * h + 2 * p + 1] = d[3];
                }
            }
        }
    }

    // Swap the warp bits with the top WB chunk-slot bits through shared memory
    // (layout A -> B when FROM_A, else B -> A) and finish those stages in registers.
    template <bool FROM_A>
    static __device__ __forceinline__ void exchange_and_top(float (&v)[NT][8], float* xbuf, int w, int lane,
                                                            int barrier_id) {
        if constexpr (Geo::WB > 0) {
#pragma unroll
            for (int idx = 0; idx < NT; ++idx) {
                const int c = chunk_of<Geo, !FROM_A>(w, idx);
                float4* p = reinterpret_cast<float4*>(xbuf + c * 256 + lane * 4);
                p[0] = make_float4(v[idx][0], v[idx][1], v[idx][2], v[idx][3]);
                p[32] = make_float4(v[idx][4], v[idx][5], v[idx][6], v[idx][7]);
            }
            named_barrier(barrier_id, Geo::GROUP_THREADS);
#pragma unroll
            for (int idx = 0; idx < NT; ++idx) {
                const int c = chunk_of<Geo, FROM_A>(w, idx);
                const float4* p = reinterpret_cast<const float4*>(xbuf + c * 256 + lane * 4);
                const float4 q0 = p[0], q1 = p[32];
                v[idx][0] = q0.x; v[idx][1] = q0.y; v[idx][2] = q0.z; v[idx][3] = q0.w;
                v[idx][4] = q1.x; v[idx][5] = q1.y; v[idx][6] = q1.z; v[idx][7] = q1.w;
            }
#pragma unroll
            for (int bit = Geo::NREST; bit < NT; bit <<= 1) {
#pragma unroll
                for (int idx = 0; idx < NT; ++idx) {
                    if ((idx & bit) == 0) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float lo = v[idx][e], hi = v[idx + bit][e];
                            v[idx][e] = lo + hi;
                            v[idx + bit][e] = lo - hi;
                        }
                    }
                }
            }
        }
    }
};

// 8 parameters at a column offset, widened to fp32
__device__ __forceinline__ void load_params8(const float* __restrict__ p, float (&v)[8]) { load8(p, v); }
__device__ __forceinline__ void load_params8(const __nv_bfloat16* __restrict__ p, float (&v)[8]) { load8(p, v); }

__device__ __forceinline__ void unpack8(const uint4& q, float (&v)[8]) {
    v[0] = bf16lo_to_f32(q.x); v[1] = bf16hi_to_f32(q.x);
    v[2] = bf16lo_to_f32(q.y); v[3] = bf16hi_to_f32(q.y);
    v[4] = bf16lo_to_f32(q.z); v[5] = bf16hi_to_f32(q.z);
    v[6] = bf16lo_to_f32(q.w); v[7] = bf16hi_to_f32(q.w);
}

// ---- forward -------------------------------------------------------------------
template <int LOGD, int TB, int RG, typename TP>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS)
mma_fwd_kernel(const __nv_bfloat16* x, const TP* __restrict__ a, const TP* __restrict__ b,
               __nv_bfloat16* y, long long T, float inv_sqrt_d) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    using X = MmaXform<Geo>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    float* xbuf = smem + rg * Geo::XCHG_FLOATS;
    uint32_t hf[4];
    make_h16_fragment(hf, lane);

    int parity = 0;
    const long long stride = static_cast<long long>(gridDim.x) * RG;
    for (long long row = static_cast<long long>(blockIdx.x) * RG + rg; row < T; row += stride) {
        const uint4* src = reinterpret_cast<const uint4*>(x + row * Geo::D);
        uint4 raw[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) raw[t] = __ldcs(src + chunk_of<Geo, false>(w, t) * 32 + lane);
        float m[NT][2][4];
        float v[NT][8];
        X::pass1_raw(raw, m, hf);
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::template exchange_and_top<true>(v, xbuf + parity * Geo::D, w, lane, 1 + rg);
        parity ^= 1;
        uint4* dst = reinterpret_cast<uint4*>(y + row * Geo::D);
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            float as[8], bs[8];
            load_params8(a + (c * 32 + lane) * 8, as);
            load_params8(b + (c * 32 + lane) * 8, bs);
            uint4 o;
            o.x = pack_bf16x2(fmaf(v[idx][0] * inv_sqrt_d, as[0], bs[0]), fmaf(v[idx][1] * inv_sqrt_d, as[1], bs[1]));
            o.y = pack_bf16x2(fmaf(v[idx][2] * inv_sqrt_d, as[2], bs[2]), fmaf(v[idx][3] * inv_sqrt_d, as[3], bs[3]));
            o.z = pack_bf16x2(fmaf(v[idx][4] * inv_sqrt_d, as[4], bs[4]), fmaf(v[idx][5] * inv_sqrt_d, as[5], bs[5]));
            o.w = pack_bf16x2(fmaf(v[idx][6] * inv_sqrt_d, as[6], bs[6]), fmaf(v[idx][7] * inv_sqrt_d, as[7], bs[7]));
            __stcs(dst + c * 32 + lane, o);
        }
    }
}

// ---- backward ------------------------------------------------------------------
// partials layout: [gridDim.x][2][D] fp32 as in the butterfly family (slot 0 holds
// sum_t dy (.) (x H) without the 1/sqrt(d) factor, slot 1 holds sum_t dy).
template <int LOGD, int TB, int RG, typename TP>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS)
mma_bwd_kernel(const __nv_bfloat16* dy, const __nv_bfloat16* x, const TP* __restrict__ a,
               __nv_bfloat16* dx, float* __restrict__ partials, long long T, float inv_sqrt_d) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    using X = MmaXform<Geo>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    float* xbuf = smem + rg * Geo::XCHG_FLOATS;
    uint32_t hf[4];
    make_h16_fragment(hf, lane);

    float da_acc[NT][8], db_acc[NT][8];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { da_acc[t][e] = 0.0f; db_acc[t][e] = 0.0f; }
    }

    const long long stride = static_cast<long long>(gridDim.x) * RG;
    for (long long row = static_cast<long long>(blockIdx.x) * RG + rg; row < T; row += stride) {
        const uint4* xsrc = reinterpret_cast<const uint4*>(x + row * Geo::D);
        const uint4* dysrc = reinterpret_cast<const uint4*>(dy + row * Geo::D);
        uint4 raw[NT], rawdy[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) raw[t] = __ldcs(xsrc + chunk_of<Geo, false>(w, t) * 32 + lane);
#pragma unroll
        for (int t = 0; t < NT; ++t) rawdy[t] = __ldcs(dysrc + chunk_of<Geo, true>(w, t) * 32 + lane);
        float m[NT][2][4];
        float v[NT][8];
        // u = x H, delivered in layout B
        X::pass1_raw(raw, m, hf);
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::template exchange_and_top<true>(v, xbuf, w, lane, 1 + rg);
        // da, db partial sums and g = a (.) dy, all in layout B
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            float as[8], wv[8];
            load_params8(a + (c * 32 + lane) * 8, as);
            unpack8(rawdy[idx], wv);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                da_acc[idx][e] = fmaf(wv[e], v[idx][e], da_acc[idx][e]);
                db_acc[idx][e] += wv[e];
                v[idx][e] = as[e] * wv[e];
            }
        }
        // dx = (g H)/sqrt(d): layout B in, layout A out
        X::pass1_f32(v, m, hf);
        X::mid_stages(m);
        X::pass2(m, v, hf);
        X::template exchange_and_top<false>(v, xbuf + Geo::D, w, lane, 1 + rg);
        uint4* dst = reinterpret_cast<uint4*>(dx + row * Geo::D);
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, false>(w, idx);
            uint4 o;
            o.x = pack_bf16x2(v[idx][0] * inv_sqrt_d, v[idx][1] * inv_sqrt_d);
            o.y = pack_bf16x2(v[idx][2] * inv_sqrt_d, v[idx][3] * inv_sqrt_d);
            o.z = pack_bf16x2(v[idx][4] * inv_sqrt_d, v[idx][5] * inv_sqrt_d);
            o.w = pack_bf16x2(v[idx][6] * inv_sqrt_d, v[idx][7] * inv_sqrt_d);
            __stcs(dst + c * 32 + lane, o);
        }
    }

    // fold the RG row groups of this CTA in a fixed order, then publish (layout B columns)
    float* out = partials + static_cast<size_t>(blockIdx.x) * 2 * Geo::D;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        __syncthreads();
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            float4* p = reinterpret_cast<float4*>(smem + rg * Geo::D + (c * 32 + lane) * 8);
            const float (&src)[8] = which == 0 ? da_acc[idx] : db_acc[idx];
            p[0] = make_float4(src[0], src[1], src[2], src[3]);
            p[1] = make_float4(src[4], src[5], src[6], src[7]);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < Geo::D; j += Geo::THREADS) {
            float s = 0.0f;
#pragma unroll
            for (int r = 0; r < RG; ++r) s += smem[r * Geo::D + j];
            out[which * Geo::D + j] = s;
        }
    }
}

}  // namespace wht
