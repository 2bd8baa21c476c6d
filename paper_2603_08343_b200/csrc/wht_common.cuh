// Device helpers shared by the kernel families: 128-bit row access, bf16 <-> fp32.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace wht {

constexpr unsigned kFullMask = 0xffffffffu;

// ---- bf16 pair <-> fp32 (a bf16 is the upper half of an fp32 word) ----------
__device__ __forceinline__ float bf16lo_to_f32(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// round-to-nearest-even pack of two fp32 into one bf16x2 word (lo = first element)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ---- 8 contiguous elements <-> 8 fp32 registers ------------------------------
__device__ __forceinline__ void load8(const float* __restrict__ p, float (&v)[8]) {
    const float4 q0 = __ldg(reinterpret_cast<const float4*>(p));
    const float4 q1 = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w;
    v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* __restrict__ p, float (&v)[8]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    v[0] = bf16lo_to_f32(q.x); v[1] = bf16hi_to_f32(q.x);
    v[2] = bf16lo_to_f32(q.y); v[3] = bf16hi_to_f32(q.y);
    v[4] = bf16lo_to_f32(q.z); v[5] = bf16hi_to_f32(q.z);
    v[6] = bf16lo_to_f32(q.w); v[7] = bf16hi_to_f32(q.w);
}
__device__ __forceinline__ void store8(float* __restrict__ p, const float (&v)[8]) {
    reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* __restrict__ p, const float (&v)[8]) {
    uint4 q;
    q.x = pack_bf16x2(v[0], v[1]);
    q.y = pack_bf16x2(v[2], v[3]);
    q.z = pack_bf16x2(v[4], v[5]);
    q.w = pack_bf16x2(v[6], v[7]);
    *reinterpret_cast<uint4*>(p) = q;
}

// three in-register butterfly stages (strides 1, 2, 4) on 8 contiguous elements
__device__ __forceinline__ void bfly8(float (&v)[8]) {
#pragma unroll
    for (int s = 1; s < 8; s <<= 1) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if ((i & s) == 0) {
                const float lo = v[i], hi = v[i + s];
                v[i] = lo + hi;
                v[i + s] = lo - hi;
            }
        }
    }
}

// ---- programmatic dependent launch ------------------------------------------------
// A kernel launched with the "programmatic stream serialization" attribute may be
// scheduled while the kernel before it in the stream is still running: its CTAs
// take SMs as they become free and run their set-up.  grid_dependency_wait() then
// blocks until that earlier kernel has completed and its writes are visible; no
// global memory may be read or written before it.  grid_launch_dependents() lets
// the kernel AFTER this one start in the same way.  Both are no-ops in a kernel
// launched without the attribute / followed by a kernel launched without it.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Column-sharded (tensor-parallel) calls: one device pointer per rank's block.
constexpr int kTpMaxRanks = 8;
struct TpParts {
    const void* p[kTpMaxRanks];
};

constexpr __host__ __device__ int ilog2_c(int v) { return v <= 1 ? 0 : 1 + ilog2_c(v >> 1); }
constexpr __host__ __device__ int imin_c(int a, int b) { return a < b ? a : b; }
constexpr __host__ __device__ int imax_c(int a, int b) { return a > b ? a : b; }

}  // namespace wht
