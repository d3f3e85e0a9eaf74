/* A plain C99 consumer of include/ekv.h: proves the header is valid C and that the library's host-side calls
 * (block pool, controller, status strings) work from a program that knows nothing of CUDA or Python.
 * Built and run by tests/test_abi.py; prints "ok" and exits 0 when every check holds. */
#include <stdio.h>
#include <string.h>

#include "ekv.h"

#define CHECK(cond)                                                       \
    do {                                                                  \
        if (!(cond)) {                                                    \
            printf("check failed at line %d: %s\n", __LINE__, #cond);     \
            return 1;                                                     \
        }                                                                 \
    } while (0)

int main(void) {
    ekv_blockpool_t *bp = NULL;
    ekv_blockpool_stats_t st;
    int32_t ids[8], from[8], to[8];
    int64_t in_use = -1, n = -1;
    ekv_controller_t *ctrl = NULL;
    ekv_controller_desc_t cd;
    int i;

    CHECK(strcmp(ekv_status_string(EKV_OK), "EKV_OK") == 0);
    CHECK(strcmp(ekv_status_string(EKV_ERR_TIMEOUT), "EKV_ERR_TIMEOUT") == 0);

    /* 4 base + 4 elastic blocks: base ids first, elastic ids only while admitted */
    CHECK(ekv_blockpool_create(4, 4, &bp) == EKV_OK);
    CHECK(ekv_blockpool_alloc(bp, 5, ids) == EKV_ERR_OOM);          /* gated: only 4 base ids exist */
    CHECK(ekv_blockpool_alloc(bp, 3, ids) == EKV_OK);
    for (i = 0; i < 3; ++i) CHECK(ids[i] == i);
    CHECK(ekv_blockpool_admit_elastic(bp) == EKV_OK);
    CHECK(ekv_blockpool_alloc(bp, 3, ids + 3) == EKV_OK);            /* last base id, then two elastic ids */
    CHECK(ids[3] == 3 && ids[4] >= 4 && ids[5] >= 4);
    CHECK(ekv_blockpool_free(bp, ids, 2) == EKV_OK);                 /* ids 0 and 1 return to the base list */
    CHECK(ekv_blockpool_gate_elastic(bp, &in_use) == EKV_OK && in_use == 2);
    CHECK(ekv_blockpool_drain_plan(bp, from, to, 8, &n) == EKV_OK && n == 2);
    for (i = 0; i < 2; ++i) CHECK(from[i] >= 4 && to[i] < 4);
    CHECK(ekv_blockpool_drain_commit(bp) == EKV_OK);
    CHECK(ekv_blockpool_stats(bp, &st) == EKV_OK);
    CHECK(st.elastic_in_use == 0 && st.admitted == 0 && st.num_gpu_blocks == 4 && st.free_base == 0);
    CHECK(ekv_blockpool_destroy(bp) == EKV_OK);

    /* controller: decommit at once when a prefill is coming, commit after a quiet window */
    cd.commit_after_decode_steps = 2;
    cd.reserve_prefill_tokens = 1000;
    CHECK(ekv_controller_create(&cd, 1, &ctrl) == EKV_OK);
    CHECK(ekv_controller_decide(ctrl, 5000) == EKV_ACT_DECOMMIT);
    CHECK(ekv_controller_decide(ctrl, 0) == EKV_ACT_NONE);
    CHECK(ekv_controller_decide(ctrl, 0) == EKV_ACT_COMMIT);
    CHECK(ekv_controller_destroy(ctrl) == EKV_OK);

    /* NULL handling never crashes */
    CHECK(ekv_pool_destroy(NULL) == EKV_OK);
    CHECK(ekv_attn_workspace_bytes(NULL, 1, 1) == 0);
    CHECK(ekv_poll_status(NULL) == EKV_ERR_INVALID && strlen(ekv_last_error()) > 0);
    printf("ok\n");
    return 0;
}
