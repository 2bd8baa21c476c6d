// Second pass of the backward, gradient sums and the copy yardstick: launchers.
#include "host_common.h"
#include "misc_kernels.cuh"

namespace wht_host {

using namespace wht;

int launch_finalize(const float* parts, int nparts, int d, float scale, float* da, float* db, cudaStream_t s,
                    int groups) {
    if (d >= 32) {
        launch_overlapped(dadb_finalize32_kernel, dim3(2 * d / 32, groups), 1024, 0, s, parts, nparts, d, scale, da, db);
    } else {
        launch_overlapped(dadb_finalize_kernel, dim3((2 * d + 255) / 256, groups), 256, 0, s, parts, nparts, d, scale,
                          da, db);
    }
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

int launch_copy_rows(const void* src, void* dst, long long n16, int sms, cudaStream_t s) {
    copy_rows_kernel<<<capped_grid(ceil_div(n16, 256), sms, 8), 256, 0, s>>>(static_cast<const uint4*>(src),
                                                                            static_cast<uint4*>(dst), n16);
    WHT_CUDA_TRY(cudaGetLastError());
    return WHT_OK;
}

}  // namespace wht_host
