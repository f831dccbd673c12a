/* A C99 translation unit that uses the library through its public header only: checks that the
 * header is valid C (not just C++), that the host-only entry points behave, and that a cache cannot
 * be created without a device-side arena. Exit code 0 = all checks passed. */
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "speca.h"

#define CHECK(cond)                                                   \
    do {                                                              \
        if (!(cond)) {                                                \
            fprintf(stderr, "check failed: %s (line %d)\n", #cond, __LINE__); \
            return 1;                                                 \
        }                                                             \
    } while (0)

int main(void) {
    speca_entry_desc_t entries[2];
    speca_cache_config_t cfg;
    size_t bytes = 0, bytes0 = 0;
    speca_cache_t* cache = NULL;

    entries[0].tokens = 4096;
    entries[0].dim = 3072;
    entries[1].tokens = 512;
    entries[1].dim = 3072;
    memset(&cfg, 0, sizeof cfg);
    cfg.n_entries = 2;
    cfg.entries = entries;
    cfg.batch = 1;
    cfg.max_order = 2;
    cfg.dtype = SPECA_BF16;
    cfg.basis = SPECA_BASIS_TAYLOR;
    cfg.verify_entry = -1;
    cfg.path = SPECA_PATH_AUTO;

    CHECK(speca_cache_arena_bytes(&cfg, &bytes) == SPECA_OK);
    CHECK(bytes >= (size_t)3 * 2 * (4096 + 512) * 3072);          /* three planes of bf16 per element */
    CHECK(bytes < (size_t)3 * 2 * (4096 + 512) * 3072 + (1u << 20));
    cfg.max_order = 0;
    CHECK(speca_cache_arena_bytes(&cfg, &bytes0) == SPECA_OK && bytes0 < bytes);
    cfg.max_order = SPECA_MAX_ORDER + 1;
    CHECK(speca_cache_arena_bytes(&cfg, &bytes) == SPECA_ERR_SHAPE);
    cfg.max_order = 2;
    CHECK(speca_cache_arena_bytes(NULL, &bytes) == SPECA_ERR_INVALID_ARG);
    CHECK(speca_cache_create(&cfg, &cache) != SPECA_OK && cache == NULL); /* no arena given */

    CHECK(fabs(speca_tau(0.3, 0.5, 50.0, 50.0) - 0.3) < 1e-15);          /* tau_T = tau0 */
    CHECK(fabs(speca_tau(0.3, 0.5, 0.0, 50.0) - 0.15) < 1e-15);          /* tau_0 = tau0 * beta */
    CHECK(speca_tau(0.3, 0.5, 1.0, 0.0) != speca_tau(0.3, 0.5, 1.0, 0.0)); /* NaN for T <= 0 */
    CHECK(strcmp(speca_status_string(SPECA_OK), "ok") == 0);
    CHECK(strstr(speca_version(), "sm_100a") != NULL);
    CHECK(speca_cache_destroy(NULL) == SPECA_OK);
    {
        const void* marker = SPECA_FEATURE_IN_PLACE;
        speca_cache_config_t zero;
        memset(&zero, 0, sizeof zero);
        CHECK(marker != NULL && zero.layout == SPECA_LAYOUT_TABLES);   /* a zeroed config asks for the paper's tables */
        CHECK(speca_cache_next_slot(NULL, 0, 0, NULL) == SPECA_ERR_INVALID_ARG);
    }
    {
        speca_cache_stats_t st;
        CHECK(sizeof st == (8 + 2 * SPECA_MAX_BATCH) * sizeof(uint64_t));   /* the binding mirrors this layout */
        CHECK(speca_cache_stats(NULL, &st) == SPECA_ERR_INVALID_ARG);
    }
    CHECK(speca_cache_update_forecast(NULL, NULL, NULL, NULL, NULL, NULL, NULL, NULL, NULL, NULL) == SPECA_ERR_INVALID_ARG);
    CHECK(speca_cache_update_forecast_multi(NULL, NULL, NULL, NULL, 2, NULL, NULL, NULL, NULL, NULL, NULL) == SPECA_ERR_INVALID_ARG);
    CHECK(speca_cache_check(NULL, NULL) == SPECA_ERR_INVALID_ARG);
    CHECK(speca_verify_decide(SPECA_METRIC_L2, NULL, 1, NULL, 0.f, NULL, NULL, NULL, NULL) == SPECA_ERR_INVALID_ARG);
    CHECK(speca_verify_pred_static(NULL, NULL, 8, 1, SPECA_BF16, NULL, 0.f, NULL, NULL, NULL, 0, NULL) ==
          SPECA_ERR_INVALID_ARG);
    printf("abi ok\n");
    return 0;
}
