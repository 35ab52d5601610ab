/* Plain C99 user of include/loma.h: proves that the header compiles as C, that the library links
 * from C, and that the host-side entry points (which make no CUDA call) behave as documented. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "loma.h"

#define CHECK(cond)                                                        \
    do {                                                                   \
        if (!(cond)) {                                                     \
            fprintf(stderr, "abi_check: failed at line %d: %s\n", __LINE__, #cond); \
            return 1;                                                      \
        }                                                                  \
    } while (0)

int main(void) {
    /* Fig. 5 geometry: t = 2, c = 2, three chunks of 10 rows */
    enum { N = 3, C = 2, T = 2, S = 30 };
    int32_t chunk[S], zone[S], offset[S], src[S], pos[S];
    uint8_t counts[S * S], by_key[S * S];
    int i, ones = 0;

    CHECK(loma_version() >= 100);
    CHECK(strstr(loma_status_string(LOMA_OK), "LOMA_OK") != NULL);
    CHECK(loma_layout_index(N, C, T, 0, 0, chunk, zone, offset, src, pos, 0, NULL) == LOMA_OK);
    CHECK(chunk[0] == 0 && zone[0] == LOMA_ZONE_READ && pos[0] == 0);
    CHECK(zone[4] == LOMA_ZONE_MEM && src[4] == -1 && pos[4] == 1);        /* Eq. 14: y*tc + (j+1)c - 1 */
    CHECK(zone[5] == LOMA_ZONE_MEM && pos[5] == 3);
    CHECK(zone[6] == LOMA_ZONE_REP && src[6] == 0);
    CHECK(chunk[29] == 2 && zone[29] == LOMA_ZONE_REP && offset[29] == 3);
    CHECK(loma_layout_index(-1, C, T, 0, 0, chunk, NULL, NULL, NULL, NULL, 0, NULL) == LOMA_ERR_INVALID_ARG);

    CHECK(loma_masked_attn_plan_coverage(N, C, T, 0, 0, counts) == LOMA_OK);
    CHECK(loma_masked_attn_bwd_plan_coverage(N, C, T, 0, 0, by_key) == LOMA_OK);
    for (i = 0; i < S * S; ++i) {
        CHECK(counts[i] <= 1 && counts[i] == by_key[i]);
        ones += counts[i];
    }
    CHECK(ones == 126);                                                     /* allowed entries of the Fig. 5 mask */

    /* argument checks happen before any CUDA call: these never touch a device */
    CHECK(loma_masked_attn_fwd((void*)0x1000, (void*)0x2000, (void*)0x3000, (void*)0x4000, NULL, 1, 1, 96, 1, 2, 2, 4, 0,
                               640, 640, 64, LOMA_BF16, 0.0f, 0u, NULL) == LOMA_ERR_UNSUPPORTED);
    CHECK(loma_decode_workspace_bytes(32, 32, 128, 8192) > 0);
    CHECK(loma_masked_attn_bwd_workspace_bytes(4, 32, 128, 32, 4, 16, 0, 0u) >= (size_t)4 * 32 * 4608 * 4);
    puts("abi_check ok");
    return 0;
}
