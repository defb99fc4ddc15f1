/* A plain C99 client of the library: proves that include/softsync_ps.h is valid C and that the protocol
 * calls can be driven without any Python or C++ on the caller's side.  With zero parameters nothing is
 * launched, so it runs on a machine without a GPU. */
#include "softsync_ps.h"

#include <stdio.h>

#define CHECK(cond) do { if (!(cond)) { printf("failed: %s (line %d)\n", #cond, __LINE__); return 1; } } while (0)

int main(void)
{
    ps_t *ps = NULL;
    int64_t ts = -1, applied = -1, logical = -1;
    static int dummy;                       /* stands for a zero-length gradient: never dereferenced */
    ps_log_entry log[4];
    int64_t state[PS_STATE_WORDS(2)];

    CHECK(ps_create(&ps, 0, 2, 1, 0.5f, 0.0f, 0.0f, PS_MOD_INV_STALENESS) == PS_OK);
    CHECK(ps_set_option(ps, PS_OPT_FUSE_T, 2) == PS_OK);
    CHECK(ps_pull_weights(ps, NULL, &ts) == PS_OK && ts == 0);
    CHECK(ps_push_gradient(ps, 1, &dummy, 0) == PS_OK);
    CHECK(ps_push_gradient(ps, 0, &dummy, 0) == PS_READY);
    CHECK(ps_pull_weights(ps, NULL, &ts) == PS_OK && ts == 1);
    CHECK(ps_push_gradient(ps, 0, &dummy, 1) == PS_OK);
    CHECK(ps_push_gradient(ps, 1, &dummy, 0) == PS_READY);          /* staleness 1 */
    CHECK(ps_peek_state(ps, NULL, NULL, &applied, &logical) == PS_OK && applied == 0 && logical == 2);
    CHECK(ps_apply_update(ps) == 2);
    CHECK(ps_apply_update(ps) == PS_ERR_NOT_READY);
    CHECK(ps_get_update_log(ps, 0, 2, log) == PS_OK);
    CHECK(log[0].learner == 0 && log[1].learner == 1 && log[3].learner == 1 && log[3].tau == 1);
    CHECK(log[0].scale == 0.25f && log[3].update == 1);
    CHECK(ps_export_state(ps, state, PS_STATE_WORDS(2)) == PS_STATE_WORDS(2));
    CHECK(ps_destroy(ps) == PS_OK);
    CHECK(ps_destroy(ps) == PS_ERR_INVALID_ARG);
    printf("c client ok: %s\n", ps_status_string(PS_READY));
    return 0;
}
