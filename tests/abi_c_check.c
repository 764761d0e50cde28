/* Test helper (not part of the product): a plain C99 program that includes the public header,
 * takes the address of every entry point and makes two calls that need no GPU, to show that the
 * header is valid C and that the library links from C.  Built and run by tests/test_abi_and_shard.py. */
#include <stdio.h>
#include <string.h>
#include "cser.h"

int main(void) {
    typedef void (*fn_t)(void);
    const fn_t fns[] = {
        (fn_t)cser_create, (fn_t)cser_create_slab, (fn_t)cser_create_ex,
        (fn_t)cser_destroy, (fn_t)cser_set_x0, (fn_t)cser_step,
        (fn_t)cser_step_host, (fn_t)cser_read_state, (fn_t)cser_read_columns,
        (fn_t)cser_write_state, (fn_t)cser_set_lr, (fn_t)cser_debug_set_masks,
        (fn_t)cser_grbs_mask, (fn_t)cser_set_timing, (fn_t)cser_last_kernel_ms,
        (fn_t)cser_launch_count, (fn_t)cser_last_error, (fn_t)cser_step_noalloc,
        (fn_t)cser_replay_begin, (fn_t)cser_step_replayable, (fn_t)cser_replay_end,
        (fn_t)cser_create_wshard, (fn_t)cser_wshard_message_elems,
        (fn_t)cser_wshard_pack, (fn_t)cser_wshard_apply, (fn_t)cser_debug_stall_next_staged_step, (fn_t)cser_build_id,
    };
    size_t i;
    for (i = 0; i < sizeof(fns) / sizeof(fns[0]); ++i)
        if (!fns[i]) return 1;
    /* invalid arguments are rejected before any CUDA call */
    if (cser_create(0, 8, 256, 4, 4, 4, 0.1f, 0.0f, 0) != NULL) return 2;
    if (strstr(cser_last_error(), "positive") == NULL) return 3;
    if (cser_step(NULL, NULL, NULL) != CSER_ERR_INVALID) return 4;
    if (cser_launch_count(NULL) != 0) return 5;
    printf("c abi ok: %u entry points\n", (unsigned)(sizeof(fns) / sizeof(fns[0])));
    return 0;
}
