/* Compiles include/sparbit.h as plain C and exercises the host-only part of the ABI (no GPU):
 * plan creation, Algorithm 1's step variables, message expansion, error codes.  Built and run by
 * tests/test_c_abi.py.  Exit code 0 = all checks passed. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "sparbit.h"

#define CHECK(cond)                                                   \
    do {                                                              \
        if (!(cond)) {                                                \
            fprintf(stderr, "line %d: %s failed\n", __LINE__, #cond); \
            return 1;                                                 \
        }                                                             \
    } while (0)

int main(void) {
    sparbit_plan_t* plan = sparbit_plan(13, 4096);
    CHECK(plan != NULL);
    CHECK(sparbit_plan_num_steps(plan) == 4); /* ceil(log2 13) */
    CHECK(sparbit_plan_last_phase(plan) == 3);
    /* Algorithm 1 for p = 13: distances 8, 4, 2, 1; 1, 2, 3, 6 blocks; the last two steps withhold one */
    {
        const int want_d[4] = {8, 4, 2, 1}, want_n[4] = {1, 2, 3, 6}, want_ig[4] = {0, 0, 1, 1};
        int total = 0;
        for (int s = 0; s < 4; s++) {
            int d, n, ig;
            CHECK(sparbit_plan_step_info(plan, s, &d, &n, &ig) == SPARBIT_OK);
            CHECK(d == want_d[s] && n == want_n[s] && ig == want_ig[s]);
            total += n;
        }
        CHECK(total == 12); /* p - 1 blocks received per rank */
    }
    /* every message of step 1 goes 4 ranks ahead and keeps its slot */
    {
        size_t n = 0;
        CHECK(sparbit_plan_messages(plan, 1, NULL, 0, &n) == SPARBIT_OK);
        CHECK(n == 26);
        sparbit_msg* m = (sparbit_msg*)malloc(n * sizeof *m);
        CHECK(m != NULL);
        CHECK(sparbit_plan_messages(plan, 1, m, n, &n) == SPARBIT_OK);
        for (size_t i = 0; i < n; i++) {
            CHECK(m[i].phase == 1);
            CHECK(m[i].dst_rank == (m[i].src_rank + 4) % 13);
            CHECK(m[i].src_slot == m[i].dst_slot);
            CHECK(m[i].src_space == SPARBIT_SPACE_RECV && m[i].dst_space == SPARBIT_SPACE_RECV);
        }
        free(m);
    }
    CHECK(sparbit_plan_workspace_bytes(plan) == 0);
    CHECK(sparbit_plan_exec_mode(plan) == SPARBIT_EXEC_MIRROR); /* 676 KiB of receive buffers in 4 KiB blocks: a cluster of CTAs */
    {
        uint64_t v = 0;
        CHECK(sparbit_plan_get_tunable(plan, SPARBIT_TUNE_BULK_MIN_BLOCK_BYTES, &v) == SPARBIT_OK && v == 8192);
        CHECK(sparbit_plan_set_tunable(plan, SPARBIT_TUNE_COUNT_, 1) == SPARBIT_ERR_ARG);
        CHECK(sparbit_rank_device(13, 2, SPARBIT_MAP_SEQUENTIAL, 6) == 1 && sparbit_rank_device(13, 2, SPARBIT_MAP_CYCLIC, 6) == 0);
        /* 13 ranks on 2 devices: 6 + 7 under the sequential mapping, 7 + 6 under the cyclic one */
        CHECK(sparbit_multi_rank_count(13, 2, SPARBIT_MAP_SEQUENTIAL, 0) == 6 && sparbit_multi_rank_count(13, 2, SPARBIT_MAP_CYCLIC, 0) == 7);
        CHECK(sparbit_multi_local_index(13, 2, SPARBIT_MAP_SEQUENTIAL, 6) == 0 && sparbit_multi_local_index(13, 2, SPARBIT_MAP_CYCLIC, 6) == 3);
        {
            void* bases[2] = {(void*)(1 << 20), NULL};
            /* the second device's buffers are missing; more devices than the table holds */
            CHECK(sparbit_allgather_multi_phases(plan, 2, SPARBIT_MAP_SEQUENTIAL, 0, (const void*)4096, bases, NULL, -1, 0) == SPARBIT_ERR_ARG);
            CHECK(sparbit_allgather_multi(plan, SPARBIT_MULTI_MAX_DEVICES + 1, SPARBIT_MAP_SEQUENTIAL, 0, (const void*)4096, bases, NULL, NULL, NULL) == SPARBIT_ERR_ARG);
        }
    }
    /* argument errors are found before anything touches a device */
    CHECK(sparbit_allgather(plan, NULL, NULL, NULL) == SPARBIT_ERR_ARG);
    CHECK(sparbit_allgather_steps(plan, (const void*)4096, (void*)(1 << 24), NULL, 3, 1) == SPARBIT_ERR_ARG);
    CHECK(sparbit_plan_destroy(plan) == SPARBIT_OK);

    {
        sparbit_plan_t* p = NULL;
        const size_t counts[4] = {16, 0, 48, 32};
        CHECK(sparbit_plan_create(6, 64, SPARBIT_ALGO_RECURSIVE_DOUBLING, SPARBIT_EXEC_AUTO, &p) == SPARBIT_ERR_UNSUPPORTED);
        CHECK(p == NULL);
        CHECK(sparbit_plan_create(7, 64, SPARBIT_ALGO_NEIGHBOR_EXCHANGE, SPARBIT_EXEC_AUTO, &p) == SPARBIT_ERR_UNSUPPORTED);
        CHECK(sparbit_plan_create(6, 64, SPARBIT_ALGO_BRUCK, SPARBIT_EXEC_AUTO, &p) == SPARBIT_OK);
        CHECK(sparbit_plan_workspace_bytes(p) == (size_t)6 * 6 * 64);
        CHECK(sparbit_plan_last_phase(p) == 3); /* 3 steps + the rotation */
        CHECK(sparbit_plan_destroy(p) == SPARBIT_OK);
        CHECK(sparbit_plan_create_v(4, counts, SPARBIT_ALGO_SPARBIT, SPARBIT_EXEC_AUTO, &p) == SPARBIT_OK);
        CHECK(sparbit_plan_num_steps(p) == 2);
        CHECK(sparbit_plan_destroy(p) == SPARBIT_OK);
        CHECK(sparbit_allgather_noalloc(64, 16, SPARBIT_ALGO_RING, (const void*)4096, (void*)(1 << 24), NULL) == SPARBIT_ERR_LIMIT);
    }
    CHECK(strcmp(sparbit_strerror(SPARBIT_OK), "success") == 0);
    CHECK(strlen(sparbit_last_cuda_error()) == 0);
    printf("abi ok\n");
    return 0;
}
