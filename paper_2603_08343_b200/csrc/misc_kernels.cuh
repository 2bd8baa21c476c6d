// Small kernels outside the kernel families: the second pass of the backward (sum of the per-CTA
// partial column sums in a fixed order), and the copy yardstick of the benchmark.
#pragma once
#include "wht_common.cuh"

namespace wht {

// ---- second pass of the backward, parallel over slices of the partials -------------
// block = 32 columns x 32 slices; slice s adds partials s, s+32, ... in order, then
// the 32 slice sums are added in order: a fixed association, bit-reproducible.
__global__ void __launch_bounds__(1024)
dadb_finalize32_kernel(const float* __restrict__ partials, int nparts, int d, float inv_sqrt_d,
                       float* __restrict__ da, float* __restrict__ db) {
    __shared__ float red[32][33];
    grid_dependency_wait();  // the partials come from the kernel launched just before
    grid_launch_dependents();
    {   // block-diagonal form: blockIdx.y is the channel group; its partials, da and db follow the group before
        partials += static_cast<size_t>(blockIdx.y) * nparts * 2 * d;
        da += static_cast<size_t>(blockIdx.y) * d;
        db += static_cast<size_t>(blockIdx.y) * d;
    }
    const int cx = threadIdx.x & 31;
    const int sl = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + cx;  // column in [0, 2d): da columns then db columns
    const int which = j / d;
    const int col = j - which * d;
    const size_t stride = static_cast<size_t>(2) * d;
    const float* src = partials + static_cast<size_t>(which) * d + col;
    float s = 0.0f;
    for (int p = sl; p < nparts; p += 32) s += src[p * stride];
    red[sl][cx] = s;
    __syncthreads();
    if (sl == 0) {
        float t = 0.0f;
#pragma unroll
        for (int k = 0; k < 32; ++k) t += red[k][cx];
        if (which == 0) da[col] = t * inv_sqrt_d; else db[col] = t;
    }
}

// ---- second pass: da[j] = inv_sqrt_d * sum_p partials[p][0][j], db[j] likewise --
__global__ void __launch_bounds__(256)
dadb_finalize_kernel(const float* __restrict__ partials, int nparts, int d, float inv_sqrt_d,
                     float* __restrict__ da, float* __restrict__ db) {
    grid_dependency_wait();  // the partials come from the kernel launched just before
    grid_launch_dependents();
    partials += static_cast<size_t>(blockIdx.y) * nparts * 2 * d;  // channel group, as above
    da += static_cast<size_t>(blockIdx.y) * d;
    db += static_cast<size_t>(blockIdx.y) * d;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= 2 * d) return;
    const int which = j / d;
    const int col = j - which * d;
    const float* src = partials + static_cast<size_t>(which) * d + col;
    const size_t stride = static_cast<size_t>(2) * d;
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
    int p = 0;
    for (; p + 4 <= nparts; p += 4) {
        s0 += src[(p + 0) * stride];
        s1 += src[(p + 1) * stride];
        s2 += src[(p + 2) * stride];
        s3 += src[(p + 3) * stride];
    }
    for (; p < nparts; ++p) s0 += src[p * stride];
    const float s = (s0 + s1) + (s2 + s3);
    if (which == 0) da[col] = s * inv_sqrt_d; else db[col] = s;
}

// ---- bandwidth yardstick: copy rows with the forward pass's access pattern ----
// (four loads in flight per thread were tried: the same at the Training size, 5 % slower at the Prefill size)
__global__ void __launch_bounds__(256)
copy_rows_kernel(const uint4* src, uint4* dst, long long n16) {
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n16; i += stride)
        __stcs(dst + i, __ldcs(src + i));
}

}  // namespace wht
