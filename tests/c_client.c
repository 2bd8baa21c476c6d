/* A plain C99 client of the C ABI: includes only the public header and the CUDA runtime's C API, reads
 * x, a, b (float32, little endian) from a file the test wrote, runs wht_affine_fwd and wht_affine_bwd_ws on
 * device copies and writes y, dx, da, db back.  The test compares the file with the oracle.
 *   usage: c_client T d in.bin out.bin        in.bin: x[T*d] dy[T*d] a[d] b[d];  out.bin: y dx da db
 * With no arguments it only checks an argument error (no GPU needed) and exits 0. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "wht_affine.h"

#define CHECK(call)                                                                  \
    do {                                                                             \
        int rc_ = (int)(call);                                                       \
        if (rc_ != 0) { fprintf(stderr, "%s -> %d\n", #call, rc_); return 2; }       \
    } while (0)

int main(int argc, char** argv) {
    if (argc == 1) {
        float buf[64] = {0.0f};
        /* d = 12 is no power of two: rejected before any CUDA call */
        return wht_affine_fwd(buf, buf, buf, buf, 1, 12, WHT_F32, NULL) == WHT_ERR_BAD_DIM ? 0 : 1;
    }
    if (argc != 5) return 64;
    const int64_t T = atoll(argv[1]);
    const int32_t d = atoi(argv[2]);
    const size_t n = (size_t)T * (size_t)d;
    const size_t in_floats = 2 * n + 2 * (size_t)d, out_floats = 2 * n + 2 * (size_t)d;
    float* host = (float*)malloc((in_floats > out_floats ? in_floats : out_floats) * sizeof(float));
    FILE* f = fopen(argv[3], "rb");
    if (!host || !f || fread(host, sizeof(float), in_floats, f) != in_floats) return 3;
    fclose(f);
    float *x, *dy, *a, *b, *y, *dx, *da, *db;
    void* ws;
    const size_t ws_bytes = wht_affine_bwd_workspace_bytes(T, d, WHT_F32);
    CHECK(cudaMalloc((void**)&x, n * 4)); CHECK(cudaMalloc((void**)&dy, n * 4));
    CHECK(cudaMalloc((void**)&y, n * 4)); CHECK(cudaMalloc((void**)&dx, n * 4));
    CHECK(cudaMalloc((void**)&a, d * 4)); CHECK(cudaMalloc((void**)&b, d * 4));
    CHECK(cudaMalloc((void**)&da, d * 4)); CHECK(cudaMalloc((void**)&db, d * 4));
    CHECK(cudaMalloc(&ws, ws_bytes ? ws_bytes : 16));
    CHECK(cudaMemcpy(x, host, n * 4, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(dy, host + n, n * 4, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(a, host + 2 * n, d * 4, cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(b, host + 2 * n + d, d * 4, cudaMemcpyHostToDevice));
    cudaStream_t s;
    CHECK(cudaStreamCreate(&s));
    CHECK(wht_affine_fwd(x, a, b, y, T, d, WHT_F32, s));
    CHECK(wht_affine_bwd_ws(dy, x, a, dx, da, db, T, d, WHT_F32, ws, ws_bytes, s));
    CHECK(cudaStreamSynchronize(s));
    CHECK(wht_affine_device_status());
    CHECK(cudaMemcpy(host, y, n * 4, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(host + n, dx, n * 4, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(host + 2 * n, da, d * 4, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(host + 2 * n + d, db, d * 4, cudaMemcpyDeviceToHost));
    f = fopen(argv[4], "wb");
    if (!f || fwrite(host, sizeof(float), out_floats, f) != out_floats) return 4;
    fclose(f);
    CHECK(wht_affine_shutdown());
    return 0;
}
