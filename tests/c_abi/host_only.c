/* A plain C consumer of the library: compiled as strict C99 against include/lagkv.h and
 * linked to the shared object.  It only makes host-side calls (a plan with device = -1), so it
 * runs without a GPU.  Prints "ok" and returns 0 when every check holds. */
#include <stdio.h>
#include <string.h>

#include "lagkv.h"

static int fail(const char *what)
{
    fprintf(stderr, "c_abi: %s\n", what);
    return 1;
}

int main(void)
{
    lagkv_config cfg;
    lagkv_plan_t plan = NULL;
    int32_t info[6];

    memset(&cfg, 0, sizeof cfg); /* zeroed: contiguous strides, LagKV scoring, bf16 */
    cfg.B = 32;
    cfg.H_kv = 8;
    cfg.D = 128;
    cfg.sink = 16;
    cfg.lag = 2048;
    cfg.keep_ratio = 0.125;
    cfg.std_ddof = 1;
    cfg.device = -1; /* host-only plan */
    if (lagkv_plan(&cfg, &plan) != LAGKV_OK || plan == NULL) return fail("lagkv_plan");
    if (lagkv_keep_count(plan) != 256) return fail("keep count");
    /* Eq. 12 at the long-context configuration: 16 + 256*62 + 2048 + 2032 */
    if (lagkv_compressed_len(plan, 131072, -1) != 19968) return fail("Eq. 12");
    if (lagkv_compressed_len(plan, 16 + 2 * 2048 - 1, -1) != 16 + 2 * 2048 - 1) return fail("skip rule");
    if (lagkv_workspace_bytes(plan, 0) == 0 || (lagkv_workspace_bytes(plan, 0) % 256) != 0) return fail("workspace");
    if (lagkv_host_staging_bytes(plan, 131072, 4) == 0 || lagkv_host_staging_bytes(plan, 131072, 33) != 0)
        return fail("staging bytes");
    if (lagkv_launch_info(plan, 131072, info) != LAGKV_OK || info[0] != 148 || info[3] != 1) return fail("launch info");
    /* a host-only plan refuses to launch */
    if (lagkv_compress_prefill(plan, (const void *)256, (const void *)512, 131072, NULL, NULL, NULL, NULL,
                               (void *)1024, 256, NULL) != LAGKV_EINVAL)
        return fail("host-only plan launched");
    lagkv_plan_destroy(plan);

    cfg.D = 80; /* no kernel for this head_dim */
    if (lagkv_plan(&cfg, &plan) != LAGKV_EUNSUPPORTED || plan != NULL) return fail("unsupported head_dim");
    if (strcmp(lagkv_status_string(LAGKV_OK), "ok") != 0) return fail("status string");
    if (lagkv_keep_for_target(16384, 16, 128, 0.5) < 1) return fail("keep for target");
    if (strstr(lagkv_version(), "sm_100a") == NULL) return fail("version");
    puts("ok");
    return 0;
}
