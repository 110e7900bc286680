/* Exercises the entry points of libef that need no GPU (layout arithmetic, argument checks,
 * error strings) from plain C.  The test builds the library's host code and this file with
 * -fsanitize=address,undefined and fails on any report.  Prints "ok". */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ef.h"

int main(void) {
    const int64_t sizes[] = {1, 3, 31, 33, 4095, 4096, 4097, 16384, 16385, 100000, 7, 128};
    const int nb = (int)(sizeof(sizes) / sizeof(sizes[0]));
    for (int B = 1; B <= nb; ++B) {
        int64_t* off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(B + 1));   /* exactly B+1 entries */
        off[0] = 0;
        for (int b = 0; b < B; ++b) off[b + 1] = off[b] + sizes[b];
        for (int M = 1; M <= 33; M += 8) {
            const uint32_t flag_sets[] = {0u, EF_FLAG_HOST_STAGING, EF_FLAG_WEIGHT_DECAY | EF_FLAG_DIAGNOSTICS,
                                          EF_FLAG_ONE_LOCAL_WORKER, EF_FLAG_FUSED_SCALE, EF_FLAG_SERVER_NO_BULK};
            for (unsigned f = 0; f < sizeof(flag_sets) / sizeof(flag_sets[0]); ++f) {
                size_t bytes = 0;
                if (ef_workspace_bytes(off[B], B, off, M, flag_sets[f], &bytes) != EF_OK || bytes == 0) return 1;
            }
        }
        size_t bytes = 0;
        if (ef_workspace_bytes(off[B] + 1, B, off, 1, 0, &bytes) != EF_ERR_INVALID_ARG) return 2;
        if (ef_workspace_bytes(off[B], B, off, 0, 0, &bytes) != EF_ERR_INVALID_ARG) return 3;
        if (ef_workspace_bytes(off[B], B, off, 1, EF_FLAG_FUSED_SCALE | EF_FLAG_SPLIT_SCALE, &bytes) !=
            EF_ERR_INVALID_ARG) return 4;
        ef_ctx* ctx = (ef_ctx*)1;
        /* argument checks come before any use of the device */
        if (ef_init(&ctx, off[B], B, off, 2, 1.5f, 0.1f, 0, (void*)256, (size_t)1 << 40, NULL) != EF_ERR_INVALID_ARG ||
            ctx != NULL) return 5;
        if (ef_init(&ctx, off[B], B, off, 2, 0.9f, 0.1f, 0, NULL, 0, NULL) != EF_ERR_WORKSPACE) return 6;
        if (ef_topk_workspace_bytes(off[B], &bytes) != EF_OK || bytes == 0) return 7;
        free(off);
    }
    for (int s = -1; s < 16; ++s)
        if (strlen(ef_strerror(s)) == 0) return 8;
    if (ef_server_step(NULL) != EF_ERR_INVALID_ARG || ef_worker_step(NULL, 0, NULL) != EF_ERR_INVALID_ARG ||
        ef_num_words(NULL) != -1 || ef_params(NULL) != NULL || ef_destroy(NULL) != EF_OK ||
        ef_message_units(NULL, 0, 1) != -1 || ef_check_status(NULL) != EF_ERR_INVALID_ARG) return 9;
    printf("ok\n");
    return 0;
}
