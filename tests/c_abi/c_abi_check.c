/* A plain C consumer of the library: shows that include/quantpipe.h compiles as C and that
 * the whole path can be driven without Python - device memory from the CUDA runtime, every
 * step through the C ABI.  Build (see tests/test_c_abi.py):
 *
 *   gcc -std=c99 -Wall -Werror -Iinclude -I$CUDA/include tests/c_abi/c_abi_check.c \
 *       -Lpaper_2211_04515_b200 -lquantpipe -L$CUDA/lib64 -lcudart -lm -o c_abi_check
 *
 * Run with no argument it only touches host-side entry points (no GPU needed) and prints
 * "host ok".  Run with "gpu" it quantizes a small ramp + noise tensor at 4 bits with the
 * directed search and at 8 bits without, sends it through pack and unpack, and checks that
 * every reconstruction lies within half a quantization step of the clamped input (the
 * defining property of the uniform quantizer, Sec. 3), then prints "gpu ok".  Exit code 0
 * on success, 1 with a message otherwise. */
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "quantpipe.h"

#define CHECK(cond, what)                                             \
    do {                                                              \
        if (!(cond)) {                                                \
            fprintf(stderr, "FAILED: %s (line %d)\n", what, __LINE__); \
            return 1;                                                 \
        }                                                             \
    } while (0)

static int host_checks(void)
{
    qp_qparams_t q;
    int32_t bits = 0;
    const int32_t allowed[] = {16, 8, 6, 4, 2};
    CHECK(qp_packed_bytes(1000, 3) == 384, "packed bytes: 3000 bits = 375 bytes, padded to 16");
    CHECK(qp_packed_bytes(10, 9) == 0, "9 bits is not a supported width");
    CHECK(fabs(qp_aciq_F(4, QP_DIST_LAPLACE) - 5.03) < 0.01, "F(4 bits), Laplace");
    CHECK(qp_make_qparams(-1.0, 1.0, 2, &q) == QP_OK && q.bits == 2 && fabsf(q.scale - 2.0f / 3.0f) < 1e-6f,
          "4 levels over [-1, 1]");
    CHECK(qp_make_qparams(1.0, 1.0, 2, &q) == QP_WARN_DEGENERATE && q.flags == 1, "empty range");
    /* 1e6 elements in 0.1 s over 100 Mbit/s: 10 bits per element fit, 8 is the widest allowed one below */
    CHECK(qp_select_bits(100e6, 0.1, 1000000, 0, allowed, 5, &bits) == QP_OK && bits == 8, "widest width that fits");
    CHECK(qp_policy_use_ds(4) == 1 && qp_policy_use_ds(8) == 0, "search at 4 bits and below");
    CHECK(strlen(qp_status_string(QP_ERR_UNSUPPORTED_BITS)) > 0, "status text");
    return 0;
}

static int gpu_round_trip(qp_ctx* ctx, const float* h_x, float* d_x, size_t n, int bits, int use_ds)
{
    const uint64_t nbytes = qp_packed_bytes(n, bits);
    void *d_packed = NULL, *d_y = NULL;
    qp_qparams_t* d_qp = NULL;
    qp_qparams_t q;
    float* h_y = (float*)malloc(n * sizeof(float));
    size_t i;
    CHECK(h_y != NULL, "malloc");
    CHECK(cudaMalloc(&d_packed, nbytes) == cudaSuccess && cudaMalloc(&d_y, n * sizeof(float)) == cudaSuccess &&
              cudaMalloc((void**)&d_qp, sizeof *d_qp) == cudaSuccess,
          "cudaMalloc");
    CHECK(qp_sender_device(ctx, d_x, QP_F32, n, bits, use_ds, QP_B_MAD, QP_DEFAULT_STEPS, QP_DEFAULT_HIST_BINS,
                           d_packed, nbytes, d_qp, NULL, NULL) == QP_OK,
          qp_last_error(ctx));
    CHECK(qp_unpack_dequantize(ctx, d_packed, n, bits, d_qp, 1, d_y, QP_F32, NULL) == QP_OK, qp_last_error(ctx));
    CHECK(cudaMemcpy(h_y, d_y, n * sizeof(float), cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(&q, d_qp, sizeof q, cudaMemcpyDeviceToHost) == cudaSuccess,
          "copy back");
    CHECK(qp_get_status(ctx, NULL) == 0, "device status word");
    CHECK(q.bits == bits && q.hi > q.lo && q.scale > 0.0f, "quantizer");
    for (i = 0; i < n; ++i) {
        const float t = h_x[i] < q.lo ? q.lo : (h_x[i] > q.hi ? q.hi : h_x[i]);
        if (fabsf(h_y[i] - t) > 0.5f * q.scale * 1.0001f + 1e-6f) {
            fprintf(stderr, "FAILED: element %zu: x %g clamped %g reconstructed %g step %g\n", i, h_x[i], t, h_y[i],
                    q.scale);
            return 1;
        }
    }
    cudaFree(d_packed);
    cudaFree(d_y);
    cudaFree(d_qp);
    free(h_y);
    return 0;
}

int main(int argc, char** argv)
{
    if (host_checks()) return 1;
    if (argc < 2 || strcmp(argv[1], "gpu") != 0) {
        printf("host ok\n");
        return 0;
    }
    {
        const size_t sizes[2] = {50000, 3000000};      /* one cooperative launch; the kernel chain */
        size_t s;
        qp_ctx* ctx = NULL;
        CHECK(qp_create(0, &ctx) == QP_OK, "qp_create");
        for (s = 0; s < 2; ++s) {
            const size_t n = sizes[s];
            float* h_x = (float*)malloc(n * sizeof(float));
            float* d_x = NULL;
            unsigned state = 12345u;
            size_t i;
            CHECK(h_x != NULL, "malloc");
            for (i = 0; i < n; ++i) {                  /* a ramp plus a little noise: any spread-out data will do */
                state = state * 1664525u + 1013904223u;
                h_x[i] = (float)i / (float)n - 0.5f + ((float)(state >> 8) / 16777216.0f - 0.5f) * 0.3f;
            }
            CHECK(cudaMalloc((void**)&d_x, n * sizeof(float)) == cudaSuccess, "cudaMalloc");
            CHECK(cudaMemcpy(d_x, h_x, n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess, "copy in");
            if (gpu_round_trip(ctx, h_x, d_x, n, 4, 1)) return 1;
            if (gpu_round_trip(ctx, h_x, d_x, n, 8, 0)) return 1;
            cudaFree(d_x);
            free(h_x);
        }
        CHECK(qp_launch_count(ctx) > 0, "kernels were launched");
        CHECK(qp_destroy(ctx) == QP_OK, "qp_destroy");
    }
    printf("gpu ok\n");
    return 0;
}
