/*
 * A plain C99 client of the library, compiled by gcc in the CPU test suite: shows that include/cocodc.h is a
 * C header (no C++ or CUDA types in any signature) and that libcocodc.so can be linked and called without
 * Python.  Only host-side calls are made, so it runs on a machine without a GPU.
 */
#include <stdio.h>
#include <string.h>

#include "cocodc.h"

int main(void)
{
    int64_t N = 0, h = 0;
    /* Section 4.1's setting: gamma = 0.4, H = 100, K = 4, Tc/Ts = 0.2 => 8 synchronisations per H (Eq. 8), h = 12 (Eq. 9) */
    cocodc_status s = cocodc_sync_budget(4, 100, 0.4, 1.0, 5.0, &N, &h);
    if (s != COCODC_OK || N != 8 || h != 12) {
        printf("sync_budget: status %d N %lld h %lld\n", (int)s, (long long)N, (long long)h);
        return 1;
    }
    if (cocodc_sync_budget(0, 100, 0.4, 1.0, 5.0, &N, &h) != COCODC_ERR_INVALID_ARG) return 2;
    if (strcmp(cocodc_status_string(COCODC_OK), "ok") != 0) return 3;

    /* a partition whose two segments overlap is refused before any device is touched */
    {
        const int32_t ptr[3] = {0, 1, 2};
        const int64_t off[2] = {0, 8};
        const int64_t len[2] = {16, 16};
        cocodc_partition part;
        cocodc_ctx *ctx = (cocodc_ctx *)&part;   /* any non-null value: it must come back null */
        part.N = 64; part.K = 2; part.n_segments = 2;
        part.frag_seg_ptr = ptr; part.seg_offset = off; part.seg_len = len;
        if (cocodc_create(&ctx, &part, 4, 0) != COCODC_ERR_INVALID_ARG || ctx != NULL) return 4;
    }
    if (cocodc_destroy(NULL) != COCODC_OK) return 5;
    if (cocodc_launch_count(NULL) != 0) return 6;
    if (cocodc_poll_status(NULL, NULL) != COCODC_ERR_INVALID_ARG) return 7;
    printf("abi client ok: N=%lld h=%lld\n", (long long)N, (long long)h);
    return 0;
}
