/* Plain-C consumer of include/remp.h: proves the header is valid C and the planner is callable without Python
 * or a GPU (remp_plan_create makes no CUDA call). Compiled and run by tests/test_library_host.py. */
#include <stdio.h>
#include <stdlib.h>

#include "remp.h"

int main(void) {
    remp_topo src = {4, 2, NULL}, dst = {8, 1, NULL};
    remp_model_shape m = {80, 8, 128, 16, 2};
    int32_t fake_lens[1] = {0}, fake_tab[1] = {0};
    remp_block_tables bt = {1, 1, fake_lens, fake_tab}; /* never dereferenced by the planner */
    remp_plan* plan = NULL;
    if (remp_plan_create(&src, &dst, &m, &bt, &plan) != REMP_OK) {
        fprintf(stderr, "plan: %s\n", remp_last_error());
        return 1;
    }
    int32_t n = remp_plan_num_items(plan);
    int32_t* items = (int32_t*)malloc(sizeof(int32_t) * 5 * (size_t)n);
    if (remp_plan_get_items(plan, items) != REMP_OK) return 2;
    /* TP4PP2 -> TP8PP1 on 8 heads: every destination rank takes its one head from source rank t/2 of the
     * stage that holds the layer: 8 items per layer */
    if (n != 80 * 8) return 3;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t* it = items + 5 * i;
        int32_t layer = it[2], h = it[3];
        if (it[4] != h + 1 || it[1] != h || it[0] != (layer / 40) * 4 + h / 2) return 4;
    }
    int64_t r = 0, w = 0;
    if (remp_plan_traffic(plan, 6059, &r, &w) != REMP_OK || r != w || r != 6059LL * 80 * 2 * 8 * 4096) return 5;
    remp_topo bad = {3, 1, NULL};
    remp_plan* none = NULL;
    if (remp_plan_create(&bad, &dst, &m, &bt, &none) != REMP_ERR_INVALID_TOPOLOGY || none != NULL) return 6;
    if (remp_shard_bytes(&dst, &m, 7, 10) != 80LL * 2 * 10 * 1 * 4096) return 7;
    free(items);
    remp_plan_destroy(plan);
    printf("c abi ok: %d items\n", n);
    return 0;
}
