/* Plain C user of libssd_sgd.so: no Python, no torch.  Replays the first hand-computed trace
 * (tests/golden/trace_wd0_K2_k2.txt: K=2, lr=0.5, m=0.5, W=1, k=2, lr_local=2, alpha=2, beta=0.5)
 * through ssd_step on device buffers from cudaMalloc and compares the final state with the
 * hand-computed values, which are exact in binary32.  Exit code 0 = all equal. */
#include <stdio.h>
#include <string.h>
#include <cuda_runtime_api.h>
#include "ssd_sgd.h"

#define N 4
#define K 2
#define CHECK(x) do { if ((x) != 0) { printf("failed: %s (line %d)\n", #x, __LINE__); return 2; } } while (0)

static int same(const char *what, const float *dev, const float *expect)
{
    float host[N];
    if (cudaMemcpy(host, dev, sizeof host, cudaMemcpyDeviceToHost) != cudaSuccess) return 0;
    if (memcmp(host, expect, sizeof host) != 0) {
        printf("%s: got %g %g %g %g\n", what, host[0], host[1], host[2], host[3]);
        return 0;
    }
    return 1;
}

int main(void)
{
    const float w0[N] = {1, -2, 0.5f, 4};
    const float grads[5][K][N] = {
        {{0.25f, 1, -0.5f, 0}, {0.75f, -1, -1.5f, 2}},
        {{0.5f, 0.25f, 1, -1}, {0, 0.75f, -1, -3}},
        {{0.25f, -0.5f, 0, 1}, {0.25f, 0.5f, 2, 1}},
        {{0, 1, -1, 0.5f}, {0, 0, 1, -0.5f}},
        {{1, 0, 0.5f, -2}, {-1, 0.5f, 0.5f, 0}}};
    /* state after iteration 4 (a pull iteration) */
    const float w_end[N] = {0.0625f, -2.96875f, 0.34375f, 4.53125f};
    const float mom_end[N] = {-0.0625f, -0.28125f, -0.34375f, 0.46875f};
    const float w_dev_end[K][N] = {{-4.125f, -8.65625f, 4.78125f, 9.59375f}, {3.875f, -4.65625f, -7.21875f, 7.59375f}};
    const float pre_end[N] = {0.25f, -2.375f, 0.875f, 4.125f};

    float *w, *mom, *w_loc[K], *pre[K], *w_dev[K], *g[K];
    CHECK(cudaMalloc((void **)&w, 256)); CHECK(cudaMalloc((void **)&mom, 256));
    for (int i = 0; i < K; ++i) {
        CHECK(cudaMalloc((void **)&w_loc[i], 256)); CHECK(cudaMalloc((void **)&pre[i], 256));
        CHECK(cudaMalloc((void **)&w_dev[i], 256)); CHECK(cudaMalloc((void **)&g[i], 256));
        CHECK(cudaMemcpy(w_loc[i], w0, sizeof w0, cudaMemcpyHostToDevice));
    }
    CHECK(cudaMemcpy(w, w0, sizeof w0, cudaMemcpyHostToDevice));
    CHECK(cudaMemset(mom, 0, 256));

    const int64_t numel[1] = {N};
    ssd_layout layout = {1, numel};
    ssd_hparams hp = {K, 0.5f, 0.5f, 0.0f, 1, 2, 2.0f, 2.0f, 0.5f, 0.5f, SSD_F32, SSD_LOCAL_GLU};
    ssd_buffers bufs = {w, mom, w_loc, pre, w_dev};
    ssd_ctx *ctx = NULL;
    int64_t padded = 0;
    CHECK(ssd_arena_numel(&layout, &padded));
    if (padded != N) return 3;
    CHECK(ssd_init(&ctx, &layout, &hp, &bufs));
    for (int n = 0; n < 5; ++n) {
        const void *gp[K];
        for (int i = 0; i < K; ++i) {
            CHECK(cudaMemcpy(g[i], grads[n][i], sizeof grads[n][i], cudaMemcpyHostToDevice));
            gp[i] = g[i];
        }
        ssd_status st = ssd_step(ctx, gp, NULL);
        if (st != SSD_OK) { printf("ssd_step: %s (%s)\n", ssd_status_str(st), ssd_last_cuda_error(ctx)); return 4; }
    }
    CHECK(cudaDeviceSynchronize());
    int64_t iter = 0, loc_update = 0;
    int32_t view = -1;
    CHECK(ssd_get_counters(ctx, &iter, &loc_update, NULL, NULL));
    CHECK(ssd_worker_weights(ctx, 0, NULL, &view));
    int ok = iter == 5 && loc_update == 4 && view == SSD_VIEW_DEVICE && ssd_kernel_launches(ctx) == 5;
    ok = ok && same("w", w, w_end) && same("mom", mom, mom_end);
    for (int i = 0; i < K; ++i)
        ok = ok && same("w_loc", w_loc[i], w_end) && same("w_dev", w_dev[i], w_dev_end[i]) && same("pre", pre[i], pre_end);
    ssd_destroy(ctx);
    printf(ok ? "trace reproduced from C\n" : "MISMATCH\n");
    return ok ? 0 : 1;
}
