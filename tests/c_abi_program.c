/* A plain C user of libcartpole.so: no Python, no C++, only cartpole.h and the CUDA runtime for the
 * caller-owned buffers. Prints what it computed as text; tests/test_zy_c_program.py compiles it,
 * runs it on the GPU and compares the numbers with the CPU oracle.
 *
 *   usage: c_abi_program n_envs T seed
 */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "cartpole.h"

#define CHECK_CP(call)                                                          \
    do {                                                                        \
        int rc_ = (call);                                                       \
        if (rc_ != CP_OK) {                                                     \
            fprintf(stderr, "%s failed (%d): %s\n", #call, rc_, cp_last_error()); \
            return 2;                                                           \
        }                                                                       \
    } while (0)
#define CHECK_CUDA(call)                                                        \
    do {                                                                        \
        cudaError_t e_ = (call);                                                \
        if (e_ != cudaSuccess) {                                                \
            fprintf(stderr, "%s failed: %s\n", #call, cudaGetErrorString(e_));   \
            return 3;                                                           \
        }                                                                       \
    } while (0)

int main(int argc, char **argv)
{
    if (argc != 4) {
        fprintf(stderr, "usage: %s n_envs T seed\n", argv[0]);
        return 1;
    }
    const int64_t n = atoll(argv[1]), T = atoll(argv[2]);
    const uint32_t seed = (uint32_t)strtoul(argv[3], NULL, 10);

    /* per-step path: a library-owned batch stepped in place three times */
    cp_state *batch = cp_reset(n, seed);
    if (!batch) {
        fprintf(stderr, "cp_reset: %s\n", cp_last_error());
        return 2;
    }
    float *d_reward;
    uint8_t *d_done;
    CHECK_CUDA(cudaMalloc((void **)&d_reward, (size_t)n * sizeof(float)));
    CHECK_CUDA(cudaMalloc((void **)&d_done, (size_t)n));
    uint32_t done_count[3];
    uint8_t *h_done = (uint8_t *)malloc((size_t)n);
    for (int k = 0; k < 3; ++k) {
        CHECK_CP(cp_step(batch, NULL, batch, d_reward, d_done));
        CHECK_CUDA(cudaMemcpy(h_done, d_done, (size_t)n, cudaMemcpyDeviceToHost));
        done_count[k] = 0;
        for (int64_t i = 0; i < n; ++i) done_count[k] += h_done[i];
    }
    uint32_t t_now;
    CHECK_CP(cp_state_info(batch, NULL, NULL, NULL, &t_now, NULL, NULL));

    /* rollout path */
    float *d_ret;
    uint32_t *d_cnt;
    uint64_t *d_tot;
    CHECK_CUDA(cudaMalloc((void **)&d_ret, (size_t)n * sizeof(float)));
    CHECK_CUDA(cudaMalloc((void **)&d_cnt, (size_t)n * sizeof(uint32_t)));
    CHECK_CUDA(cudaMalloc((void **)&d_tot, 2 * sizeof(uint64_t)));
    CHECK_CUDA(cudaMemset(d_tot, 0, 2 * sizeof(uint64_t)));
    cp_returns ret;
    memset(&ret, 0, sizeof ret);
    ret.ep_return_sum = d_ret;
    ret.ep_count = d_cnt;
    ret.totals = d_tot;
    CHECK_CP(cp_rollout(n, T, seed, NULL, &ret));
    float *h_ret = (float *)malloc((size_t)n * sizeof(float));
    uint64_t h_tot[2];
    CHECK_CUDA(cudaMemcpy(h_ret, d_ret, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(h_tot, d_tot, sizeof h_tot, cudaMemcpyDeviceToHost));

    /* a bad call is refused with a message, not a crash */
    const int bad = cp_rollout(n, 0, seed, NULL, &ret);

    printf("version %s\n", cp_version());
    printf("t %u\n", t_now);
    printf("done_counts %u %u %u\n", done_count[0], done_count[1], done_count[2]);
    printf("totals %llu %llu\n", (unsigned long long)h_tot[0], (unsigned long long)h_tot[1]);
    printf("returns");
    for (int64_t i = 0; i < n && i < 16; ++i) printf(" %.0f", h_ret[i]);
    printf("\n");
    printf("bad_call %d %s\n", bad, cp_last_error());

    cp_free(batch);
    cp_shutdown();
    cudaFree(d_reward);
    cudaFree(d_done);
    cudaFree(d_ret);
    cudaFree(d_cnt);
    cudaFree(d_tot);
    free(h_done);
    free(h_ret);
    return 0;
}
