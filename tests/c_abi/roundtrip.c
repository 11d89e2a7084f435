/* A plain C caller of libkvq: no Python, no torch.  Reads x (16-bit patterns) and lambda (fp32) from files, runs
 * kvq_encode and kvq_decode on device buffers it allocates itself, and writes signs, packed codes, scales and the
 * reconstruction back to files for the test to compare with the oracle.
 *
 *   roundtrip D N dtype(0 = fp16, 1 = bf16) n_lambda rows_per_lambda seed dir
 */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "kvq.h"

static void *slurp(const char *dir, const char *name, size_t bytes)
{
    char path[1024];
    snprintf(path, sizeof path, "%s/%s", dir, name);
    FILE *f = fopen(path, "rb");
    void *p = malloc(bytes);
    if (!f || !p || fread(p, 1, bytes, f) != bytes) {
        fprintf(stderr, "cannot read %zu bytes from %s\n", bytes, path);
        exit(2);
    }
    fclose(f);
    return p;
}

static void dump(const char *dir, const char *name, const void *p, size_t bytes)
{
    char path[1024];
    snprintf(path, sizeof path, "%s/%s", dir, name);
    FILE *f = fopen(path, "wb");
    if (!f || fwrite(p, 1, bytes, f) != bytes) {
        fprintf(stderr, "cannot write %s\n", path);
        exit(2);
    }
    fclose(f);
}

#define CK(call)                                                                         \
    do {                                                                                 \
        kvq_status_t st_ = (call);                                                       \
        if (st_ != KVQ_OK) {                                                             \
            fprintf(stderr, "%s -> %s\n", #call, kvq_status_string(st_));                \
            return 1;                                                                    \
        }                                                                                \
    } while (0)
#define CU(call)                                                                         \
    do {                                                                                 \
        cudaError_t e_ = (call);                                                         \
        if (e_ != cudaSuccess) {                                                         \
            fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_));                \
            return 1;                                                                    \
        }                                                                                \
    } while (0)

int main(int argc, char **argv)
{
    if (argc != 8) {
        fprintf(stderr, "usage: roundtrip D N dtype n_lambda rows_per_lambda seed dir\n");
        return 2;
    }
    const int D = atoi(argv[1]);
    const long long N = atoll(argv[2]);
    const kvq_dtype_t dtype = atoi(argv[3]) ? KVQ_BF16 : KVQ_F16;
    const long long n_lambda = atoll(argv[4]), rpl = atoll(argv[5]);
    const unsigned long long seed = strtoull(argv[6], NULL, 10);
    const char *dir = argv[7];
    const int group = 32;
    const size_t xb = (size_t)N * D * 2, pb = (size_t)N * D / 2, sb = (size_t)N * (D / group) * 2, lb = (size_t)n_lambda * D * 4;

    void *hx = slurp(dir, "x.bin", xb), *hl = slurp(dir, "lambda.bin", lb);
    void *dx, *dl, *dp, *ds, *dout;
    CU(cudaMalloc(&dx, xb));
    CU(cudaMalloc(&dl, lb));
    CU(cudaMalloc(&dp, pb));
    CU(cudaMalloc(&ds, sb));
    CU(cudaMalloc(&dout, xb));
    CU(cudaMemcpy(dx, hx, xb, cudaMemcpyHostToDevice));
    CU(cudaMemcpy(dl, hl, lb, cudaMemcpyHostToDevice));

    kvq_plan_t *plan = NULL;
    CK(kvq_plan_create(D, group, seed, &plan));
    int8_t signs[512];
    CK(kvq_plan_get_signs(plan, signs));
    CK(kvq_encode(plan, dx, dtype, N, (const float *)dl, n_lambda, rpl, (uint8_t *)dp, ds, NULL));
    CK(kvq_decode(plan, (const uint8_t *)dp, ds, N, (const float *)dl, n_lambda, rpl, dout, dtype, NULL));
    uint32_t word = 0;
    CK(kvq_plan_device_status(plan, &word));
    CU(cudaDeviceSynchronize());

    void *hp = malloc(pb), *hs = malloc(sb), *ho = malloc(xb);
    CU(cudaMemcpy(hp, dp, pb, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(hs, ds, sb, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(ho, dout, xb, cudaMemcpyDeviceToHost));
    dump(dir, "signs.bin", signs, (size_t)D);
    dump(dir, "packed.bin", hp, pb);
    dump(dir, "scales.bin", hs, sb);
    dump(dir, "out.bin", ho, xb);
    CK(kvq_plan_destroy(plan));
    printf("ok launches=%llu status_word=%u\n", (unsigned long long)kvq_launch_count(), word);
    return 0;
}
