/* A plain C99 consumer of include/forge.h: compiled with -std=c99 -Wall -Wextra -Werror
 * -pedantic and linked against libforge.so by tests/test_boundary_cpu.py.  It exercises the
 * host-only entry points (plan query, strings, NULL-argument paths); no GPU is needed. */
#include <stdio.h>
#include <string.h>

#include "forge.h"

static int failures = 0;
#define CHECK(cond)                                                         \
    do {                                                                    \
        if (!(cond)) {                                                      \
            fprintf(stderr, "line %d: %s\n", __LINE__, #cond);              \
            ++failures;                                                     \
        }                                                                   \
    } while (0)

int main(void)
{
    forge_fused_linear_desc_t d;
    forge_plan_info_t info;
    forge_fused_linear_t h = NULL;
    int detail[4] = {0, 0, 0, 0};
    double rate = 0.0;

    memset(&d, 0, sizeof d);
    d.M = 8192; d.N = 8192; d.K = 8192;
    d.dtype = FORGE_BF16; d.act = FORGE_ACT_SILU; d.red = FORGE_RED_NONE;
    d.scale = 1.0f; d.ln_eps = 1e-5f; d.has_bias = 1; d.device = 0;

    CHECK(forge_fused_linear_query_plan(&d, 148, &info) == FORGE_OK);
    CHECK(info.kernel == FORGE_KERNEL_BF16_TCGEN05);
    CHECK(info.cluster == 2 && info.tile_m == 256 && info.tile_n == 256);
    CHECK(strstr(forge_kernel_name(info.kernel), "tcgen05") != NULL);

    d.M = 16; d.red = FORGE_RED_MAX;
    CHECK(forge_fused_linear_query_plan(&d, 148, &info) == FORGE_OK);
    CHECK(info.kernel == FORGE_KERNEL_BF16_SKINNY);

    d.K = 12;                                   /* 16-bit rows need a 16-byte pitch */
    CHECK(forge_fused_linear_query_plan(&d, 148, &info) == FORGE_ERR_UNSUPPORTED);
    d.K = 0;
    CHECK(forge_fused_linear_query_plan(&d, 148, &info) == FORGE_ERR_INVALID_ARG);

    CHECK(forge_fused_linear_query_plan(NULL, 148, &info) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_query_plan(&d, 148, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_create(NULL, &h) == FORGE_ERR_INVALID_ARG && h == NULL);
    CHECK(forge_fused_linear_create(&d, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_run(NULL, NULL, NULL, NULL, NULL, NULL, NULL, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_run_host(NULL, NULL, NULL, NULL, NULL, NULL, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_last_status(NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_last_wait_detail(NULL, detail) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_get_plan(NULL, &info) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_launches_per_run(NULL) == 0);
    CHECK(forge_fused_linear_destroy(NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(strcmp(forge_fused_linear_kernel_name(NULL), "no handle") == 0);
    CHECK(forge_selftest_bounded_wait(0, 0, detail) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_selftest_ffma_rate(0, 0, &rate, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_selftest_ffma_rate(0, 10, NULL, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_selftest_read_stream(0, NULL, NULL) == FORGE_ERR_INVALID_ARG);
    CHECK(forge_fused_linear_f32_reduce_static(0, 1, 1, FORGE_ACT_RELU, FORGE_RED_SUM, 1.0f, NULL, NULL, NULL, NULL,
                                               NULL) == FORGE_ERR_INVALID_ARG);

    CHECK(strcmp(forge_status_string(FORGE_OK), "ok") == 0);
    CHECK(strcmp(forge_status_string((forge_status_t)99), "unknown status") == 0);
    CHECK(strcmp(forge_kernel_name((forge_kernel_t)99), "unknown kernel") == 0);
    CHECK(FORGE_STATIC_SCRATCH_BYTES == 1048576u);

    if (failures == 0) printf("forge.h as C99: ok\n");
    return failures == 0 ? 0 : 1;
}
