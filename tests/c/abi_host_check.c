/* Compiled as plain C99 against include/ws.h and linked with libws.so: checks that the header is
 * valid C and exercises the host-only entry points (no GPU needed).  Prints the segment table of
 * the worked example of Section 4.1 ([3,3,256,256] with 8, 10 and 64 shards) and of Section 5.2
 * (a 4 MB tensor cut 2048 ways).  Exit code 0 = every check passed. */
#include <stdio.h>
#include <string.h>

#include "ws.h"

static int check(int cond, const char* what) {
    if (!cond) fprintf(stderr, "FAILED: %s\n", what);
    return cond ? 0 : 1;
}

int main(void) {
    int bad = 0;
    ws_tensor_desc d[2];
    ws_plan* plan = NULL;
    const ws_segment* segs = NULL;
    int32_t T = 0;
    const int shards[3] = {8, 10, 64};
    int i;

    memset(d, 0, sizeof(d));
    d[0].ndim = 4;
    d[0].dims[0] = 3; d[0].dims[1] = 3; d[0].dims[2] = 256; d[0].dims[3] = 256;
    for (i = 0; i < 3; ++i) {
        bad += check(ws_plan_create(d, 1, shards[i], 8, 0, &plan) == WS_OK, "ws_plan_create");
        bad += check(ws_plan_segments(plan, &segs, &T) == WS_OK && T == 1, "ws_plan_segments");
        printf("[3,3,256,256] R=%d: piece %lld, shard %lld, padded total %lld\n", shards[i],
               (long long)segs[0].piece, (long long)ws_plan_shard_elems(plan),
               (long long)(ws_plan_shard_elems(plan) * shards[i]));
        bad += check(ws_plan_shard_elems(plan) * shards[i] <= 10LL * 256 * 256, "no more padding than [10,256,256]");
        bad += check(ws_plan_valid_elems(plan) == 589824, "valid elements");
        ws_plan_destroy(plan);
    }
    d[0].ndim = 1;
    d[0].dims[0] = 1048576;                                   /* 4 MB of fp32 */
    bad += check(ws_plan_create(d, 1, 2048, 8, 0, &plan) == WS_OK, "ws_plan_create(4MB)");
    bad += check(ws_plan_shard_elems(plan) * 4 == 2048, "4 MB / 2048 = 2 KB");
    bad += check(ws_workspace_bytes(plan, WS_ADAM) == 0 && ws_workspace_bytes(plan, WS_LAMB) > 0, "workspace sizes");
    bad += check(ws_pack(plan, NULL, WS_F32, NULL, NULL) == WS_ERR_INVALID_ARG, "null arguments are refused");
    ws_plan_destroy(plan);

    d[1].ndim = 1;
    d[1].dims[0] = 100;
    d[0].dims[0] = 37;
    bad += check(ws_plan_create_layout(d, 2, 4, 8, 0, WS_LAYOUT_CONCAT, &plan) == WS_OK, "concatenated layout");
    bad += check(ws_plan_layout(plan) == WS_LAYOUT_CONCAT && ws_plan_shard_elems(plan) == 40, "40 + 100 in 4 shards of 40");
    ws_plan_destroy(plan);

    bad += check(ws_plan_create(d, 1, 0, 8, 0, &plan) == WS_ERR_INVALID_ARG && plan == NULL, "R = 0 is refused");
    bad += check(strcmp(ws_status_string(WS_OK), "ok") == 0, "status string");
    bad += check(ws_static_scratch_bytes() == WS_STATIC_SCRATCH_BYTES, "static scratch size");
    printf("%s\n", bad ? "FAILED" : "all host-side ABI checks passed");
    return bad ? 1 : 0;
}
