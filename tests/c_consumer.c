/*
 * A caller of the astra.h ABI written in plain C with nothing but the CUDA runtime: no Python, no
 * torch.  test_gpu_c_consumer.py writes the inputs of one call of each operation to files, runs
 * this program, and compares the files it writes back with the oracle.
 *
 * usage: c_consumer <dir> <dtype: 0 bf16 | 1 fp16 | 2 fp32> <T> <H> <D> <Hh> <Dh> <n_parts>
 *   reads  <dir>/x.bin, r.bin, w.bin                [T,H], [T,H], [H]          fused_add_rmsnorm (eps 1e-5)
 *          <dir>/silu_in.bin                        [T,2D]                     silu_and_mul
 *          <dir>/va.bin, vb.bin, sa.bin, sb.bin     [T,Hh,Dh] x2, [T,Hh] x2    merge_attn_states_lse
 *          <dir>/part<i>.bin, ar_r.bin              n_parts x [T,H], [T,H]     fused_allreduce_add_rmsnorm
 *   writes <dir>/y.bin, r_out.bin, silu_out.bin, vo.bin, so.bin, ar_y.bin, ar_r_out.bin
 * Exit code 0 on success; otherwise the number of the step that failed.
 */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "astra.h"

static int step = 0;
#define CHECK(cond)                                                       \
    do {                                                                  \
        ++step;                                                           \
        if (!(cond)) {                                                    \
            fprintf(stderr, "c_consumer: step %d failed: %s\n", step, #cond); \
            return step;                                                  \
        }                                                                 \
    } while (0)

static char path[4096];
static const char *in_dir(const char *dir, const char *name) {
    snprintf(path, sizeof path, "%s/%s", dir, name);
    return path;
}

/* device buffer filled from a file of exactly `bytes` bytes (NULL on any failure) */
static void *upload(const char *dir, const char *name, size_t bytes) {
    void *host = malloc(bytes ? bytes : 1), *dev = NULL;
    FILE *f = fopen(in_dir(dir, name), "rb");
    if (!host || !f || fread(host, 1, bytes, f) != bytes || cudaMalloc(&dev, bytes ? bytes : 1) != cudaSuccess ||
        cudaMemcpy(dev, host, bytes, cudaMemcpyHostToDevice) != cudaSuccess)
        dev = NULL;
    if (f) fclose(f);
    free(host);
    return dev;
}

static int download(const char *dir, const char *name, const void *dev, size_t bytes) {
    void *host = malloc(bytes ? bytes : 1);
    int ok = host && cudaMemcpy(host, dev, bytes, cudaMemcpyDeviceToHost) == cudaSuccess;
    FILE *f = ok ? fopen(in_dir(dir, name), "wb") : NULL;
    ok = ok && f && fwrite(host, 1, bytes, f) == bytes;
    if (f) fclose(f);
    free(host);
    return ok;
}

int main(int argc, char **argv) {
    if (argc != 9) return 100;
    const char *dir = argv[1];
    const astra_dtype_t dt = (astra_dtype_t)atoi(argv[2]);
    const int64_t T = atoll(argv[3]), H = atoll(argv[4]), D = atoll(argv[5]), Hh = atoll(argv[6]), Dh = atoll(argv[7]);
    const int n_parts = atoi(argv[8]);
    const size_t e = dt == ASTRA_FP32 ? 4 : 2;
    cudaStream_t stream;
    CHECK(cudaSetDevice(0) == cudaSuccess);
    CHECK(cudaStreamCreate(&stream) == cudaSuccess);

    /* fused_add_rmsnorm, in place */
    void *x = upload(dir, "x.bin", T * H * e), *r = upload(dir, "r.bin", T * H * e), *w = upload(dir, "w.bin", H * e);
    CHECK(x && r && w);
    CHECK(astra_fused_add_rmsnorm(x, r, w, T, H, 1e-5f, dt, stream) == ASTRA_OK);

    /* silu_and_mul */
    void *si = upload(dir, "silu_in.bin", T * 2 * D * e), *so = NULL;
    CHECK(si && cudaMalloc(&so, T * D * e) == cudaSuccess);
    CHECK(astra_silu_and_mul(so, si, T, D, dt, stream) == ASTRA_OK);

    /* merge_attn_states_lse */
    const size_t vbytes = T * Hh * Dh * e, sbytes = T * Hh * 4;
    void *va = upload(dir, "va.bin", vbytes), *vb = upload(dir, "vb.bin", vbytes), *vo = NULL;
    float *sa = (float *)upload(dir, "sa.bin", sbytes), *sb = (float *)upload(dir, "sb.bin", sbytes), *lo = NULL;
    CHECK(va && vb && sa && sb && cudaMalloc(&vo, vbytes) == cudaSuccess && cudaMalloc((void **)&lo, sbytes) == cudaSuccess);
    CHECK(astra_merge_attn_states_lse(vo, lo, va, sa, vb, sb, T, Hh, Dh, dt, stream) == ASTRA_OK);

    /* fused_allreduce_add_rmsnorm */
    const void *parts[16];
    CHECK(n_parts >= 1 && n_parts <= 16);
    for (int p = 0; p < n_parts; ++p) {
        char name[32];
        snprintf(name, sizeof name, "part%d.bin", p);
        parts[p] = upload(dir, name, T * H * e);
        CHECK(parts[p] != NULL);
    }
    void *ar_r = upload(dir, "ar_r.bin", T * H * e), *ar_y = NULL;
    CHECK(ar_r && cudaMalloc(&ar_y, T * H * e) == cudaSuccess);
    CHECK(astra_fused_allreduce_add_rmsnorm(ar_y, ar_r, parts, n_parts, w, T, H, 1e-5f, dt, stream) == ASTRA_OK);

    /* argument errors come back as codes, and an empty batch is fine, with a GPU present too */
    CHECK(astra_silu_and_mul(so, so, T, D, dt, stream) == ASTRA_ERR_OVERLAP);
    CHECK(astra_fused_add_rmsnorm(NULL, NULL, NULL, 0, H, 1e-5f, dt, stream) == ASTRA_OK);

    CHECK(cudaStreamSynchronize(stream) == cudaSuccess);
    CHECK(cudaGetLastError() == cudaSuccess);
    CHECK(download(dir, "y.bin", x, T * H * e) && download(dir, "r_out.bin", r, T * H * e));
    CHECK(download(dir, "silu_out.bin", so, T * D * e));
    CHECK(download(dir, "vo.bin", vo, vbytes) && download(dir, "so.bin", lo, sbytes));
    CHECK(download(dir, "ar_y.bin", ar_y, T * H * e) && download(dir, "ar_r_out.bin", ar_r, T * H * e));
    printf("ok\n");
    return 0;
}
