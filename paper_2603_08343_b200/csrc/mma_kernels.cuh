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
//
// All fp32 arithmetic outside the mma is done on register pairs with the packed
// f32x2 add / fma of sm_100, which halves its issue slots.
#pragma once
#include "wht_common.cuh"

namespace wht {

using F2 = float2;

__device__ __forceinline__ F2 f2(float x, float y) { return make_float2(x, y); }
__device__ __forceinline__ F2 add2(F2 a, F2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ F2 sub2(F2 a, F2 b) { return __ffma2_rn(b, f2(-1.0f, -1.0f), a); }  // a - b, exact product
__device__ __forceinline__ F2 mul2(F2 a, F2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ void bfly2(F2& lo, F2& hi) {
    const F2 s = add2(lo, hi);
    hi = sub2(lo, hi);
    lo = s;
}
__device__ __forceinline__ F2 unpack_bf16x2(uint32_t u) { return f2(bf16lo_to_f32(u), bf16hi_to_f32(u)); }
__device__ __forceinline__ uint32_t pack_bf16x2(F2 v) { return pack_bf16x2(v.x, v.y); }

// D(16x8, fp32) += A(16x16, bf16) * B(16x8, bf16); d01 = (c0, c1), d23 = (c2, c3)
__device__ __forceinline__ void mma_bf16_m16n8k16(F2& d01, F2& d23, const uint32_t (&a)[4], uint32_t b0,
                                                  uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d01.x), "+f"(d01.y), "+f"(d23.x), "+f"(d23.y)
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

// fp32 pair -> bf16x2 hi (round to nearest) and bf16x2 lo (rounded remainder):
// hi + lo carries the pair to a relative error of 2^-17.
__device__ __forceinline__ void split_hi_lo(F2 v, uint32_t& hi, uint32_t& lo) {
    hi = pack_bf16x2(v);
    lo = pack_bf16x2(sub2(v, unpack_bf16x2(hi)));
}

// fp32 pair -> three bf16x2 terms hi + mid + lo: 24 significant bits, i.e. the fp32 value itself (up to
// the exponent range of bf16, which is fp32's).
__device__ __forceinline__ void split_hi_mid_lo(F2 v, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
    hi = pack_bf16x2(v);
    const F2 r = sub2(v, unpack_bf16x2(hi));
    mid = pack_bf16x2(r);
    lo = pack_bf16x2(sub2(r, unpack_bf16x2(mid)));
}

// d += H_16 * [b0; b1] with the fp32 operands carried as NS bf16 terms each (NS mma into one accumulator):
// NS = 2 carries 16-17 significant bits, NS = 3 all 24.
template <int NS>
__device__ __forceinline__ void mma_split(F2& d01, F2& d23, const uint32_t (&hf)[4], F2 b0, F2 b1) {
    if constexpr (NS == 2) {
        uint32_t b0h, b0l, b1h, b1l;
        split_hi_lo(b0, b0h, b0l);
        split_hi_lo(b1, b1h, b1l);
        mma_bf16_m16n8k16(d01, d23, hf, b0h, b1h);
        mma_bf16_m16n8k16(d01, d23, hf, b0l, b1l);
    } else {
        uint32_t b0h, b0m, b0l, b1h, b1m, b1l;
        split_hi_mid_lo(b0, b0h, b0m, b0l);
        split_hi_mid_lo(b1, b1h, b1m, b1l);
        mma_bf16_m16n8k16(d01, d23, hf, b0h, b1h);
        mma_bf16_m16n8k16(d01, d23, hf, b0m, b1m);
        mma_bf16_m16n8k16(d01, d23, hf, b0l, b1l);
    }
}

__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int LOGD, int TB, int RG_>
struct MmaGeo {
    static constexpr int D = 1 << LOGD;
    static constexpr int NT = 1 << TB;         // chunks of 8 elements per thread
    static constexpr int WB = LOGD - 8 - TB;   // stages that cross warps
    static_assert(TB >= 0 && WB >= 0 && WB <= TB, "unsupported split of the row");
    static constexpr int W = 1 << WB;          // warps per row
    static constexpr int NREST = NT / W;
    static constexpr int RG = RG_;             // rows in flight per CTA
    static constexpr int GROUP_THREADS = W * 32;
    static constexpr int THREADS = RG * GROUP_THREADS;
    static constexpr int XCHG_ONE = (W - 1) * NT * 256;     // floats that change owner in one exchange
    static constexpr int XCHG_FLOATS = 2 * XCHG_ONE;        // per row group (two buffers, used alternately)
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

// Thread-local views of a row slice:
//   m[t][h][p]  (after pass 1)  pair r = (x, y) <-> index bit 5, p <-> bit 1, h <-> bit 2
//   v[t][j]     (load layout)   pair (x, y) = elements 2j, 2j+1 of chunk slot t
//   NS: bf16 terms an fp32 operand of a pass is carried as (2 for bf16 rows, 3 for fp32 rows)
template <class Geo, int NS = 2>
struct MmaXform {
    static constexpr int NT = Geo::NT;

    // pass 1 on stored bf16 (bits {0,3,4,1})
    static __device__ __forceinline__ void pass1_raw(const uint4 (&raw)[NT], F2 (&m)[NT][2][2],
                                                     const uint32_t (&hf)[4]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            m[t][0][0] = m[t][0][1] = m[t][1][0] = m[t][1][1] = f2(0.0f, 0.0f);
            mma_bf16_m16n8k16(m[t][0][0], m[t][0][1], hf, raw[t].x, raw[t].y);
            mma_bf16_m16n8k16(m[t][1][0], m[t][1][1], hf, raw[t].z, raw[t].w);
        }
    }

    // pass 1 on fp32 values in load layout (hi/lo split operands)
    static __device__ __forceinline__ void pass1_f32(const F2 (&v)[NT][4], F2 (&m)[NT][2][2],
                                                     const uint32_t (&hf)[4]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                m[t][h][0] = m[t][h][1] = f2(0.0f, 0.0f);
                mma_split<NS>(m[t][h][0], m[t][h][1], hf, v[t][2 * h + 0], v[t][2 * h + 1]);
            }
        }
    }

    // fp32 butterflies on bit 2 (h) and on chunk-slot bits 1..TB-1.  A row of one chunk per thread
    // (d = 256) has no bit 8 for pass 2, which takes bit 2 instead: nothing to do here.
    static __device__ __forceinline__ void mid_stages(F2 (&m)[NT][2][2]) {
        if constexpr (NT == 1) return;
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            bfly2(m[t][0][0], m[t][1][0]);
            bfly2(m[t][0][1], m[t][1][1]);
        }
#pragma unroll
        for (int bit = 2; bit < NT; bit <<= 1) {
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                if ((t & bit) == 0) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        bfly2(m[t][h][0], m[t + bit][h][0]);
                        bfly2(m[t][h][1], m[t + bit][h][1]);
                    }
                }
            }
        }
    }

    // pass 2 on bits {5,6,7} and chunk-slot bit 0; the result is in load layout.  With one chunk per
    // thread (d = 256) the fourth bit is bit 2 instead: the register select of the B fragment is h, and the
    // two halves of the accumulator fragment are h = 0 and h = 1 of the output.
    static __device__ __forceinline__ void pass2(const F2 (&m)[NT][2][2], F2 (&v)[NT][4],
                                                 const uint32_t (&hf)[4]) {
        if constexpr (NT == 1) {
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                F2 d01 = f2(0.0f, 0.0f), d23 = f2(0.0f, 0.0f);
                mma_split<NS>(d01, d23, hf, m[0][0][p], m[0][1][p]);
                v[0][p] = d01;
                v[0][2 + p] = d23;
            }
            return;
        }
#pragma unroll
        for (int u = 0; u < NT / 2; ++u) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    F2 d01 = f2(0.0f, 0.0f), d23 = f2(0.0f, 0.0f);
                    mma_split<NS>(d01, d23, hf, m[2 * u][h][p], m[2 * u + 1][h][p]);
                    v[2 * u][2 * h + p] = d01;
                    v[2 * u + 1][2 * h + p] = d23;
                }
            }
        }
    }

    // Swap the warp bits with the top WB chunk-slot bits through shared memory and
    // finish those stages in registers.  Slot (top, rest) of warp w moves to warp
    // `top`, slot (w, rest): a transpose of the (warp, top) grid, the same in both
    // directions (layout A -> B and B -> A); slots with top == w stay where they are
    // and are not copied.  xbuf holds XCHG_ONE floats.
    static __device__ __forceinline__ void exchange_and_top(F2 (&v)[NT][4], float* xbuf, int w, int lane,
                                                            int barrier_id) {
        if constexpr (Geo::WB > 0) {
            constexpr int W = Geo::W, NREST = Geo::NREST;
            // compact position of the block sent from warp `src` to warp `dst` (src != dst)
            auto block_of = [](int src, int dst, int rest) {
                return ((src * (W - 1) + dst - (dst > src ? 1 : 0)) * NREST + rest) * 256;
            };
#pragma unroll
            for (int idx = 0; idx < NT; ++idx) {
                const int top = idx / NREST, rest = idx % NREST;
                if (top != w) {
                    float4* p = reinterpret_cast<float4*>(xbuf + block_of(w, top, rest) + lane * 4);
                    p[0] = make_float4(v[idx][0].x, v[idx][0].y, v[idx][1].x, v[idx][1].y);
                    p[32] = make_float4(v[idx][2].x, v[idx][2].y, v[idx][3].x, v[idx][3].y);
                }
            }
            named_barrier(barrier_id, Geo::GROUP_THREADS);
#pragma unroll
            for (int idx = 0; idx < NT; ++idx) {
                const int top = idx / NREST, rest = idx % NREST;
                if (top != w) {
                    const float4* p = reinterpret_cast<const float4*>(xbuf + block_of(top, w, rest) + lane * 4);
                    const float4 q0 = p[0], q1 = p[32];
                    v[idx][0] = f2(q0.x, q0.y); v[idx][1] = f2(q0.z, q0.w);
                    v[idx][2] = f2(q1.x, q1.y); v[idx][3] = f2(q1.z, q1.w);
                }
            }
#pragma unroll
            for (int bit = NREST; bit < NT; bit <<= 1) {
#pragma unroll
                for (int idx = 0; idx < NT; ++idx) {
                    if ((idx & bit) == 0) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) bfly2(v[idx][j], v[idx + bit][j]);
                    }
                }
            }
        }
    }
};

// 8 parameters at a column offset in global memory, widened to fp32 pairs
__device__ __forceinline__ void load_params8(const float* __restrict__ p, F2 (&v)[4]) {
    const float4 q0 = __ldg(reinterpret_cast<const float4*>(p));
    const float4 q1 = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = f2(q0.x, q0.y); v[1] = f2(q0.z, q0.w);
    v[2] = f2(q1.x, q1.y); v[3] = f2(q1.z, q1.w);
}
__device__ __forceinline__ void load_params8(const __nv_bfloat16* __restrict__ p, F2 (&v)[4]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    v[0] = unpack_bf16x2(q.x); v[1] = unpack_bf16x2(q.y);
    v[2] = unpack_bf16x2(q.z); v[3] = unpack_bf16x2(q.w);
}

// Eight contiguous row elements of one thread ("chunk"), as stored: how the direct-load kernels read and
// write rows of either storage type.  `pairs` are the fp32 values as four packed pairs (elements 2j, 2j+1).
template <typename TIO> struct MmaRowIO;
template <> struct MmaRowIO<__nv_bfloat16> {
    using Raw = uint4;
    static constexpr bool kStoredBf16 = true;
    static __device__ __forceinline__ Raw load(const __nv_bfloat16* row, int chunk) {
        return __ldcs(reinterpret_cast<const uint4*>(row) + chunk);
    }
    static __device__ __forceinline__ Raw staged(const unsigned char* row, int chunk) {  // row in shared memory
        return reinterpret_cast<const uint4*>(row)[chunk];
    }
    static __device__ __forceinline__ void pairs(const Raw& r, F2 (&v)[4]) {
        v[0] = unpack_bf16x2(r.x); v[1] = unpack_bf16x2(r.y); v[2] = unpack_bf16x2(r.z); v[3] = unpack_bf16x2(r.w);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* row, int chunk, const F2 (&v)[4]) {
        uint4 o;
        o.x = pack_bf16x2(v[0]); o.y = pack_bf16x2(v[1]); o.z = pack_bf16x2(v[2]); o.w = pack_bf16x2(v[3]);
        __stcs(reinterpret_cast<uint4*>(row) + chunk, o);
    }
};
template <> struct MmaRowIO<float> {
    struct Raw { float4 a, b; };
    static constexpr bool kStoredBf16 = false;
    static __device__ __forceinline__ Raw load(const float* row, int chunk) {
        Raw r;
        r.a = __ldcs(reinterpret_cast<const float4*>(row) + 2 * chunk);
        r.b = __ldcs(reinterpret_cast<const float4*>(row) + 2 * chunk + 1);
        return r;
    }
    static __device__ __forceinline__ Raw staged(const unsigned char* row, int chunk) {
        // lanes 32 bytes apart: lanes l and l + 4 of a quarter-warp would meet in the same banks, so every
        // other group of four lanes fetches its two halves in the opposite order
        const int sw = (chunk >> 2) & 1;
        const float4 p = reinterpret_cast<const float4*>(row)[2 * chunk + sw];
        const float4 q = reinterpret_cast<const float4*>(row)[2 * chunk + (sw ^ 1)];
        Raw r;
        r.a = sw ? q : p;
        r.b = sw ? p : q;
        return r;
    }
    static __device__ __forceinline__ void pairs(const Raw& r, F2 (&v)[4]) {
        v[0] = f2(r.a.x, r.a.y); v[1] = f2(r.a.z, r.a.w); v[2] = f2(r.b.x, r.b.y); v[3] = f2(r.b.z, r.b.w);
    }
    static __device__ __forceinline__ void store(float* row, int chunk, const F2 (&v)[4]) {
        __stcs(reinterpret_cast<float4*>(row) + 2 * chunk, make_float4(v[0].x, v[0].y, v[1].x, v[1].y));
        __stcs(reinterpret_cast<float4*>(row) + 2 * chunk + 1, make_float4(v[2].x, v[2].y, v[3].x, v[3].y));
    }
};

// In every helper below `as` is a / sqrt(d): the normalisation rides on the scale
// vector, so the forward epilogue is one fma and the backward needs no final scale
// (H is linear: ((a/sqrt(d)) (.) dy) H = ((a (.) dy) H)/sqrt(d)).

// y chunk = as (.) v + b, rounded to the stored type once and stored (128-bit, streaming)
template <typename TIO>
__device__ __forceinline__ void fwd_store_chunk(const F2 (&v)[4], const F2 (&as)[4], const F2 (&bs)[4],
                                                TIO* row, int chunk) {
    F2 o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = fma2(v[j], as[j], bs[j]);
    MmaRowIO<TIO>::store(row, chunk, o);
}
// y chunk = r + (as (.) v + b) with r the 8 stored residual values `res`: the sum is taken in
// fp32 and rounded to the stored type once
template <typename TIO>
__device__ __forceinline__ void fwd_store_chunk_res(const F2 (&v)[4], const F2 (&as)[4], const F2 (&bs)[4],
                                                    const typename MmaRowIO<TIO>::Raw& res, TIO* row, int chunk) {
    F2 o[4], r[4];
    MmaRowIO<TIO>::pairs(res, r);
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = add2(fma2(v[j], as[j], bs[j]), r[j]);
    MmaRowIO<TIO>::store(row, chunk, o);
}

// the same for a bf16 chunk given by its address
__device__ __forceinline__ void fwd_store_chunk(const F2 (&v)[4], const F2 (&as)[4], const F2 (&bs)[4], uint4* dst) {
    fwd_store_chunk<__nv_bfloat16>(v, as, bs, reinterpret_cast<__nv_bfloat16*>(dst), 0);
}
__device__ __forceinline__ void fwd_store_chunk_res(const F2 (&v)[4], const F2 (&as)[4], const F2 (&bs)[4],
                                                    const uint4& res, uint4* dst) {
    fwd_store_chunk_res<__nv_bfloat16>(v, as, bs, res, reinterpret_cast<__nv_bfloat16*>(dst), 0);
}

// backward, between the two transforms, one chunk: da += dy (.) u, db += dy, v <- as (.) dy
template <typename TIO>
__device__ __forceinline__ void bwd_mid_chunk(F2 (&v)[4], const typename MmaRowIO<TIO>::Raw& rawdy,
                                              const F2 (&as)[4], F2 (&da_acc)[4], F2 (&db_acc)[4]) {
    F2 dyv[4];
    MmaRowIO<TIO>::pairs(rawdy, dyv);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        da_acc[j] = fma2(dyv[j], v[j], da_acc[j]);
        db_acc[j] = add2(db_acc[j], dyv[j]);
        v[j] = mul2(as[j], dyv[j]);
    }
}

// Fold the RG row groups' partial sums of one CTA in a fixed order and publish them.
// partials layout: [gridDim.x][2][D] fp32 (slot 0: sum_t dy (.) (x H) without the
// 1/sqrt(d) factor, slot 1: sum_t dy).  `fold` is RG*D floats of shared memory.
template <class Geo>
__device__ __forceinline__ void bwd_publish_partials(const F2 (&da_acc)[Geo::NT][4], const F2 (&db_acc)[Geo::NT][4],
                                                     float* fold, float* __restrict__ partials, int rg, int w,
                                                     int lane) {
    // block-diagonal form: the partials of channel group blockIdx.y follow those of the group before
    float* out = partials + (static_cast<size_t>(blockIdx.y) * gridDim.x + blockIdx.x) * 2 * Geo::D;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        __syncthreads();
#pragma unroll
        for (int idx = 0; idx < Geo::NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            float4* p = reinterpret_cast<float4*>(fold + rg * Geo::D + (c * 32 + lane) * 8);
            const F2 (&src)[4] = which == 0 ? da_acc[idx] : db_acc[idx];
            p[0] = make_float4(src[0].x, src[0].y, src[1].x, src[1].y);
            p[1] = make_float4(src[2].x, src[2].y, src[3].x, src[3].y);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < Geo::D; j += Geo::THREADS) {
            float s = 0.0f;
#pragma unroll
            for (int r = 0; r < Geo::RG; ++r) s += fold[r * Geo::D + j];
            out[which * Geo::D + j] = s;
        }
    }
}

// ---- forward, rows loaded straight from global memory (few rows / decode) ----------
//   TIO: storage type of the rows.  bf16 rows enter the first pass as they are (exact) and later passes as
//   two bf16 terms; fp32 rows enter every pass as three, so that no pass rounds below fp32.
template <int LOGD, int TB, int RG, typename TP, typename TIO = __nv_bfloat16>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS)
mma_fwd_kernel(const TIO* x, const TP* __restrict__ a, const TP* __restrict__ b,
               const TIO* resid, TIO* y, long long T, long long ld, float inv_sqrt_d) {
    // ld: elements between consecutive rows (>= D).  Block-diagonal form: blockIdx.y picks the channel
    // group [y*D, (y+1)*D) of rows ld wide.
    using Geo = MmaGeo<LOGD, TB, RG>;
    using IO = MmaRowIO<TIO>;
    using Raw = typename IO::Raw;
    using X = MmaXform<Geo, IO::kStoredBf16 ? 2 : 3>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    float* xbuf = smem + rg * Geo::XCHG_FLOATS;
    uint32_t hf[4];
    make_h16_fragment(hf, lane);
    const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
    {
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        x += goff; y += goff; a += goff; b += goff;
        if (resid != nullptr) resid += goff;
    }
    grid_dependency_wait();
    grid_launch_dependents();

    // With few chunks per thread (the few-rows / decode shapes) a and b are fetched once, up front,
    // so that their latency overlaps the row load instead of following the transform.
    constexpr bool PRELOAD = NT <= 4;
    F2 pas[PRELOAD ? NT : 1][4], pbs[PRELOAD ? NT : 1][4];
    if constexpr (PRELOAD) {
#pragma unroll
        for (int idx = 0; idx < NT; ++idx) {
            const int c = chunk_of<Geo, true>(w, idx);
            load_params8(a + (c * 32 + lane) * 8, pas[idx]);
            load_params8(b + (c * 32 + lane) * 8, pbs[idx]);
#pragma unroll
            for (int j = 0; j < 4; ++j) pas[idx][j] = mul2(pas[idx][j], rs2);
        }
    }

    int parity = 0;
    const long long stride = static_cast<long long>(gridDim.x) * RG;
    // Narrow rows (one or two 128-bit loads per lane and row) put little data in flight per warp, and the
    // registers allow only ~40 warps per SM: a warp requests U of its rows before it transforms the first.
    constexpr int U = (Geo::WB == 0 && NT <= 2) ? 4 / NT : 1;
    auto load_row = [&](long long r, Raw (&dst)[NT]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) dst[t] = IO::load(x + r * ld, chunk_of<Geo, false>(w, t) * 32 + lane);
    };
    for (long long row0 = static_cast<long long>(blockIdx.x) * RG + rg; row0 < T; row0 += U * stride) {
        Raw raws[U][NT];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (row0 + u * stride < T) load_row(row0 + u * stride, raws[u]);  // uniform over the warp
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long row = row0 + u * stride;
            if (row >= T) break;
            Raw res[NT];
            if (resid != nullptr) {  // the residual chunks too, ahead of the transform
#pragma unroll
                for (int idx = 0; idx < NT; ++idx)
                    res[idx] = IO::load(resid + row * ld, chunk_of<Geo, true>(w, idx) * 32 + lane);
            }
            F2 m[NT][2][2];
            F2 v[NT][4];
            if constexpr (IO::kStoredBf16) {
                X::pass1_raw(raws[u], m, hf);
            } else {
#pragma unroll
                for (int t = 0; t < NT; ++t) IO::pairs(raws[u][t], v[t]);
                X::pass1_f32(v, m, hf);
            }
            X::mid_stages(m);
            X::pass2(m, v, hf);
            X::exchange_and_top(v, xbuf + parity * Geo::XCHG_ONE, w, lane, 1 + rg);
            parity ^= 1;
            TIO* dst = y + row * ld;
#pragma unroll
            for (int idx = 0; idx < NT; ++idx) {
                const int c = chunk_of<Geo, true>(w, idx);
                F2 as[4], bs[4];
                if constexpr (PRELOAD) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) { as[j] = pas[idx][j]; bs[j] = pbs[idx][j]; }
                } else {
                    load_params8(a + (c * 32 + lane) * 8, as);
                    load_params8(b + (c * 32 + lane) * 8, bs);
#pragma unroll
                    for (int j = 0; j < 4; ++j) as[j] = mul2(as[j], rs2);
                }
                if (resid != nullptr) {
                    fwd_store_chunk_res<TIO>(v[idx], as, bs, res[idx], dst, c * 32 + lane);
                } else {
                    fwd_store_chunk<TIO>(v[idx], as, bs, dst, c * 32 + lane);
                }
            }
        }
    }
}

// ---- backward, rows loaded straight from global memory ------------------------------
template <int LOGD, int TB, int RG, typename TP, typename TIO = __nv_bfloat16>
__global__ void __launch_bounds__(MmaGeo<LOGD, TB, RG>::THREADS)
mma_bwd_kernel(const TIO* dy, const TIO* x, const TP* __restrict__ a,
               TIO* dx, float* __restrict__ partials, long long T, long long ld, float inv_sqrt_d) {
    using Geo = MmaGeo<LOGD, TB, RG>;
    using IO = MmaRowIO<TIO>;
    using Raw = typename IO::Raw;
    using X = MmaXform<Geo, IO::kStoredBf16 ? 2 : 3>;
    constexpr int NT = Geo::NT;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int rg = warp / Geo::W;
    const int w = warp % Geo::W;
    float* xbuf = smem + rg * Geo::XCHG_FLOATS;
    uint32_t hf[4];
    make_h16_fragment(hf, lane);
    const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
    {
        const long long goff = static_cast<long long>(blockIdx.y) * Geo::D;
        dy += goff; x += goff; dx += goff; a += goff;
    }

    F2 da_acc[NT][4], db_acc[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
#pragma unroll
        for (int j = 0; j < 4; ++j) { da_acc[t][j] = f2(0.0f, 0.0f); db_acc[t][j] = f2(0.0f, 0.0f); }
    }

    const long long stride = static_cast<long long>(gridDim.x) * RG;
    // A warp may request U of its rows (x and dy) before it transforms the first.  Measured: with two tensors
    // and the column sums in registers this costs occupancy and loses at every narrow width (d = 256: 0.885 ->
    // 0.73 of the copy rate, d = 512: 0.84 -> 0.61), unlike in the forward; so U = 1, the hook stays.
    constexpr int U = 1;
    auto load_rows = [&](long long r, Raw (&dx_)[NT], Raw (&ddy)[NT]) {
#pragma unroll
        for (int t = 0; t < NT; ++t) dx_[t] = IO::load(x + r * ld, chunk_of<Geo, false>(w, t) * 32 + lane);
#pragma unroll
        for (int t = 0; t < NT; ++t) ddy[t] = IO::load(dy + r * ld, chunk_of<Geo, true>(w, t) * 32 + lane);
    };
    for (long long row0 = static_cast<long long>(blockIdx.x) * RG + rg; row0 < T; row0 += U * stride) {
        Raw raws[U][NT], rawdys[U][NT];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (row0 + u * stride < T) load_rows(row0 + u * stride, raws[u], rawdys[u]);  // uniform over the warp
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long row = row0 + u * stride;
            if (row >= T) break;
            F2 m[NT][2][2];
            F2 v[NT][4];
            // u = x H, delivered in layout B
            if constexpr (IO::kStoredBf16) {
                X::pass1_raw(raws[u], m, hf);
            } else {
#pragma unroll
                for (int t = 0; t < NT; ++t) IO::pairs(raws[u][t], v[t]);
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
                load_params8(a + (c * 32 + lane) * 8, as);
#pragma unroll
                for (int j = 0; j < 4; ++j) as[j] = mul2(as[j], rs2);
                bwd_mid_chunk<TIO>(v[idx], rawdys[u][idx], as, da_acc[idx], db_acc[idx]);
            }
            // dx = (g H)/sqrt(d): layout B in, layout A out
            X::pass1_f32(v, m, hf);
            X::mid_stages(m);
            X::pass2(m, v, hf);
            X::exchange_and_top(v, xbuf + Geo::XCHG_ONE, w, lane, 1 + rg);
#pragma unroll
            for (int idx = 0; idx < NT; ++idx)
                IO::store(dx + row * ld, chunk_of<Geo, false>(w, idx) * 32 + lane, v[idx]);
        }
    }
    bwd_publish_partials<Geo>(da_acc, db_acc, smem, partials, rg, w, lane);
}

}  // namespace wht
