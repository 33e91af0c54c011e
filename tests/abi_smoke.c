/* Plain C99 client of the library's C ABI: host-only entry points, no GPU needed.
 * Compiled and run by tests/test_library_abi.py to prove the header is valid C. */
#include <math.h>
#include <stdio.h>
#include <string.h>

#include "dd_merge.h"

int main(void)
{
    double arrival[4] = {0.1, 0.5, INFINITY, 0.2};
    uint64_t mask = 0;
    int admitted = 0;
    uint64_t bits[5] = {3, 3, 2, 2, 2};
    int32_t frag[5];
    uint64_t totals[2];
    dd_grace_controller gc;
    dd_merge_record rec;

    if (dd_select_quorum(arrival, 4, 2, 0.3, &mask, &admitted) != DD_OK) return 1;
    if (mask != 0xbu || admitted != 3) return 2;
    if (dd_grace_window(2.0, 1.0, 0.25, 0.5, 0.5) != 0.625) return 3;
    if (dd_plan_fragments(bits, NULL, 5, 2, DD_FRAG_BALANCED, frag, totals) != DD_OK) return 4;
    if (totals[0] + totals[1] != 12 || (totals[0] != 7 && totals[1] != 7)) return 5;
    if (dd_grace_controller_init(&gc, 2.0, 0.5, 0.9) != DD_OK) return 6;
    if (dd_grace_controller_observe(&gc, 1.0, 0.25, 0.5) != DD_OK) return 7;
    if (dd_grace_controller_window(&gc) != 0.625) return 8;
    if (strcmp(dd_status_string(DD_OK), "ok") != 0) return 9;
    if (dd_merge_fragment(NULL, NULL, NULL, NULL, 1, DD_BF16, NULL, NULL, 0, 0, 0.7f, 0.9f, 0, 0, NULL,
                          NULL, NULL) != DD_ERR_INVALID_ARG) return 10;
    memset(&rec, 0, sizeof rec);
    printf("abi ok %zu %d\n", sizeof rec, DD_MAX_LEARNERS);
    return 0;
}
