/* The C ABI used from plain C: no Python, no torch.  Runs the hand-worked routing example
 * (R=2 T=2 K=2 E=4; ids r0t0=[2,0] r0t1=[0,3] r1t0=[0,2] r1t1=[3,2]) through layout, dispatch and
 * combine with identity experts, a 2-rank all-reduce, and a second step with the early-x promise and the
 * in-place expert stand-in, and checks the results.
 * Build: gcc c_abi_demo.c -I<include> -I<cuda>/include <libstrata_moe.so> -L<cuda>/lib64 -lcudart */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "strata_collective.h"
#include "strata_moe.h"

#define CHECK(cond)                                                        \
    do {                                                                   \
        if (!(cond)) {                                                     \
            printf("FAIL line %d: %s\n", __LINE__, #cond);                 \
            return 1;                                                      \
        }                                                                  \
    } while (0)

static uint16_t bf16_of_small_int(int v) /* exact for |v| <= 256 */
{
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

int main(void)
{
    enum { R = 2, T = 2, K = 2, E = 4, H = 8, N = R * T * K, NTOK = R * T };
    const int32_t ids[N] = {2, 0, 0, 3, 0, 2, 3, 2};
    const int32_t want_row[N] = {3, 0, 1, 6, 2, 4, 7, 5};
    const int32_t want_off[E + 1] = {0, 3, 3, 6, 8};
    const float w[N] = {0.25f, 0.75f, 0.25f, 0.75f, 0.25f, 0.75f, 0.25f, 0.75f};
    uint16_t x[NTOK * H];
    for (int n = 0; n < NTOK; ++n)
        for (int c = 0; c < H; ++c) x[n * H + c] = bf16_of_small_int(16 * (n + 1) + c);

    strata_moe_shape shape;
    memset(&shape, 0, sizeof shape);
    shape.R = R; shape.T = T; shape.H = H; shape.E = E; shape.K = K;
    shape.dispatch_dtype = STRATA_BF16;
    strata_ctx *ctx = NULL;
    CHECK(strata_ctx_create(&ctx, &shape, 0) == STRATA_OK);
    size_t ws_bytes = 0, recv_rows = 0;
    CHECK(strata_moe_workspace_bytes(&shape, &ws_bytes) == STRATA_OK && ws_bytes > 0);
    CHECK(strata_moe_recv_rows(&shape, &recv_rows) == STRATA_OK && recv_rows == N);

    void *ws, *d_ids, *d_x, *d_w, *d_recv, *d_out, *d_meta;
    CHECK(cudaMalloc(&ws, ws_bytes) == cudaSuccess);
    CHECK(cudaMalloc(&d_ids, sizeof ids) == cudaSuccess && cudaMalloc(&d_x, sizeof x) == cudaSuccess);
    CHECK(cudaMalloc(&d_w, sizeof w) == cudaSuccess && cudaMalloc(&d_recv, N * H * 2) == cudaSuccess);
    CHECK(cudaMalloc(&d_out, sizeof x) == cudaSuccess && cudaMalloc(&d_meta, 4096) == cudaSuccess);
    CHECK(strata_ctx_set_workspace(ctx, ws, ws_bytes) == STRATA_OK);
    CHECK(cudaMemcpy(d_ids, ids, sizeof ids, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(d_x, x, sizeof x, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(d_w, w, sizeof w, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemset(d_recv, 0xFF, N * H * 2) == cudaSuccess);

    int32_t *m = (int32_t *)d_meta;
    strata_moe_layout_t lay;
    memset(&lay, 0, sizeof lay);
    lay.expert_count = m;            /* [E]   */
    lay.expert_offset = m + 16;      /* [E+1] */
    lay.rank_count = m + 32;         /* [R]   */
    lay.rank_offset = m + 48;        /* [R+1] */
    lay.src_expert_count = m + 64;   /* [R,E] */
    lay.dst_row = m + 128;           /* [N]   */
    lay.src_of_row = m + 192;        /* [N]   */

    /* dispatch refuses a receive buffer nobody registered */
    CHECK(strata_moe_layout(ctx, (const int32_t *)d_ids, &lay, NULL) == STRATA_OK);
    CHECK(strata_moe_dispatch(ctx, &lay, d_x, d_recv, NULL, N, NULL) == STRATA_ERR_NOT_REGISTERED);
    uint64_t rid = 0;
    CHECK(strata_pool_register(ctx, d_recv, N * H * 2, &rid) == STRATA_OK);
    CHECK(strata_pool_is_ready(ctx, d_recv, N * H * 2) == STRATA_OK);
    CHECK(strata_moe_dispatch(ctx, &lay, d_x, d_recv, NULL, N, NULL) == STRATA_OK);
    CHECK(strata_moe_combine(ctx, &lay, d_recv, N, (const float *)d_w, d_out, NULL) == STRATA_OK);
    strata_status dev = STRATA_ERR_CUDA;
    CHECK(strata_device_status(ctx, NULL, &dev) == STRATA_OK && dev == STRATA_OK);

    int32_t got_row[N], got_off[E + 1];
    uint16_t recv[N * H], out[NTOK * H];
    CHECK(cudaMemcpy(got_row, lay.dst_row, sizeof got_row, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(got_off, lay.expert_offset, sizeof got_off, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(recv, d_recv, sizeof recv, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(cudaMemcpy(out, d_out, sizeof out, cudaMemcpyDeviceToHost) == cudaSuccess);
    CHECK(memcmp(got_row, want_row, sizeof want_row) == 0);
    CHECK(memcmp(got_off, want_off, sizeof want_off) == 0);
    for (int i = 0; i < N; ++i) CHECK(memcmp(recv + got_row[i] * H, x + (i / K) * H, H * 2) == 0);
    CHECK(memcmp(out, x, sizeof x) == 0);            /* identity experts, weights sum to 1 */

    /* all-reduce over the 2 emulated ranks: rank r holds the row r of x */
    CHECK(strata_allreduce(ctx, 2, d_x, d_out, H, NULL) == STRATA_OK);
    CHECK(strata_device_status(ctx, NULL, &dev) == STRATA_OK && dev == STRATA_OK);
    CHECK(cudaMemcpy(out, d_out, 2 * H * 2, cudaMemcpyDeviceToHost) == cudaSuccess);
    for (int c = 0; c < H; ++c) {
        const uint16_t s = bf16_of_small_int(16 + c + 32 + c);
        CHECK(out[c] == s && out[H + c] == s);
    }
    /* a second step with dispatch allowed to read x while the layout still runs, and the in-place expert stand-in
     * doubling every occupied row (x holds small integers, so 2x is exact in bf16): out = 2 x */
    float two[E], zero[E];
    for (int e = 0; e < E; ++e) { two[e] = 2.0f; zero[e] = 0.0f; }
    void *d_scale, *d_bias;
    CHECK(cudaMalloc(&d_scale, sizeof two) == cudaSuccess && cudaMalloc(&d_bias, sizeof zero) == cudaSuccess);
    CHECK(cudaMemcpy(d_scale, two, sizeof two, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(cudaMemcpy(d_bias, zero, sizeof zero, cudaMemcpyHostToDevice) == cudaSuccess);
    CHECK(strata_ctx_set_x_early(ctx, 1) == STRATA_OK);
    CHECK(strata_moe_layout(ctx, (const int32_t *)d_ids, &lay, NULL) == STRATA_OK);
    CHECK(strata_moe_dispatch(ctx, &lay, d_x, d_recv, NULL, N, NULL) == STRATA_OK);
    CHECK(strata_moe_expert_affine_inplace(ctx, &lay, d_recv, N, (const float *)d_scale, (const float *)d_bias, 2, NULL)
          == STRATA_ERR_SHAPE);                      /* packed segments: a tile is one row */
    CHECK(strata_moe_expert_affine_inplace(ctx, &lay, d_recv, N, (const float *)d_scale, (const float *)d_bias, 1, NULL)
          == STRATA_OK);
    CHECK(strata_moe_combine(ctx, &lay, d_recv, N, (const float *)d_w, d_out, NULL) == STRATA_OK);
    CHECK(strata_device_status(ctx, NULL, &dev) == STRATA_OK && dev == STRATA_OK);
    CHECK(cudaMemcpy(out, d_out, sizeof out, cudaMemcpyDeviceToHost) == cudaSuccess);
    for (int n = 0; n < NTOK; ++n)
        for (int c = 0; c < H; ++c) CHECK(out[n * H + c] == bf16_of_small_int(2 * (16 * (n + 1) + c)));
    cudaFree(d_scale); cudaFree(d_bias);

    uint64_t launches = 0;
    CHECK(strata_ctx_launch_count(ctx, &launches) == STRATA_OK && launches == 8);
    CHECK(strata_ctx_destroy(ctx) == STRATA_OK);
    cudaFree(ws); cudaFree(d_ids); cudaFree(d_x); cudaFree(d_w); cudaFree(d_recv); cudaFree(d_out); cudaFree(d_meta);
    printf("PASS %s\n", strata_status_string(STRATA_OK));
    return 0;
}
