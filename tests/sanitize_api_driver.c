/* Drives the host side of the C ABI (include/ga.h): every argument check that must answer with an
 * error code instead of touching memory. Built together with the library's source under
 * -fsanitize=address,undefined by tests/test_sanitizers.py. Without a CUDA device ga_create
 * itself fails cleanly and only the device-independent checks run; with one, the checks that need
 * an engine run as well. Exit status 0 = every call answered as expected. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ga.h"

#define EXPECT(cond)                                                        \
    do {                                                                    \
        if (!(cond)) {                                                      \
            fprintf(stderr, "line %d: %s (last error: %s)\n", __LINE__, #cond, ga_last_error()); \
            return 1;                                                       \
        }                                                                   \
    } while (0)

int main(void) {
    EXPECT(ga_last_error() != NULL);
    EXPECT(ga_create(0, 4, 0.1f, 0.9f, 0.999f, GA_GA) == NULL && strstr(ga_last_error(), "n_params"));
    EXPECT(ga_create(10, 0, 0.1f, 0.9f, 0.999f, GA_GA) == NULL);
    EXPECT(ga_create(10, 4, -1.0f, 0.9f, 0.999f, GA_GA) == NULL);
    EXPECT(ga_create(10, 4, 1e-38f, 0.9f, 0.999f, GA_GA) == NULL && strstr(ga_last_error(), "rounds to zero"));
    EXPECT(ga_create(10, 4, 0.1f, 1.0f, 0.999f, GA_GA) == NULL);
    EXPECT(ga_create(10, 4, 0.1f, 0.9f, 1.0f, GA_GA) == NULL);
    EXPECT(ga_create(10, 4, 0.1f, 0.9f, 0.999f, 99) == NULL && strstr(ga_last_error(), "variant"));
    ga_destroy(NULL);
    EXPECT(ga_push(NULL, 0, NULL) == GA_ERR_ARG);
    EXPECT(ga_pull(NULL, 0) == NULL && ga_saved(NULL, 0) == NULL);
    EXPECT(ga_push_batch(NULL, NULL, NULL, 0, NULL) == GA_ERR_ARG);
    EXPECT(ga_push_batch_host(NULL, NULL, NULL, 0, NULL, NULL) == GA_ERR_ARG);
    EXPECT(ga_get(NULL, GA_THETA, NULL) == GA_ERR_ARG && ga_gap(NULL, 0, NULL) == GA_ERR_ARG);
    EXPECT(ga_set_option(NULL, GA_OPT_STATS, 1.0) == GA_ERR_ARG && ga_set_lr(NULL, 0.1f) == GA_ERR_ARG);
    double s = 0, m = 0;
    EXPECT(ga_get_stats(NULL, &s, &m) == GA_ERR_ARG && ga_get_stats_window(NULL, &s, &m, 1) == GA_ERR_ARG);
    EXPECT(ga_export_state(NULL, NULL, 0) == 0 && ga_import_state(NULL, "x", 1) == GA_ERR_ARG);
    EXPECT(ga_num_arrivals(NULL) == GA_ERR_ARG && ga_worker_iter(NULL, 0) == GA_ERR_ARG);
    EXPECT(ga_set_layers(NULL, NULL, 1) == GA_ERR_ARG && ga_num_layers(NULL) == GA_ERR_ARG);
    /* the allocation-free call checks everything before it reaches the device */
    float* fake = (float*)(size_t)0x10000;   /* never dereferenced on the host */
    double* out = (double*)(size_t)0x20000;
    EXPECT(ga_gap_stats_noalloc(NULL, fake, fake, 16, 0.1f, 0.999f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, fake, fake, 0, 0.1f, 0.999f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, fake, fake, GA_NOALLOC_MAX_PARAMS + 1, 0.1f, 0.999f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, (float*)((size_t)fake + 4), fake, 16, 0.1f, 0.999f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, fake, fake, 16, 0.0f, 0.999f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, fake, fake, 16, 0.1f, 1.0f, 1, out, NULL) == GA_ERR_ARG);
    EXPECT(ga_gap_stats_noalloc(fake, fake, fake, 16, 0.1f, 0.999f, -1, out, NULL) == GA_ERR_ARG);

    EXPECT(ga_workspace_bytes(0, 3, GA_GA) == 0 && ga_workspace_bytes(10, 0, GA_GA) == 0 && ga_workspace_bytes(10, 3, 99) == 0);
    EXPECT(ga_workspace_bytes(1000, 3, GA_DANA_GA) > ga_workspace_bytes(1000, 3, GA_GA));
    EXPECT(ga_create_in(0, 3, 0.1f, 0.9f, 0.999f, GA_GA, fake, 1 << 20) == NULL);

    ga_engine* e = ga_create(1000, 3, 0.1f, 0.9f, 0.999f, GA_GA);
    if (!e) {   /* no CUDA device here: that must be an error message, not a crash */
        EXPECT(strlen(ga_last_error()) > 0);
        printf("sanitize api driver ok (no device: %s)\n", ga_last_error());
        return 0;
    }
    int sched[2] = {0, 7};
    const float* grads[2] = {fake, fake};
    EXPECT(ga_push_batch(e, sched, grads, 2, NULL) == GA_ERR_ARG);      /* worker 7 does not exist */
    EXPECT(ga_push_batch(e, sched, grads, -1, NULL) == GA_ERR_ARG);
    EXPECT(ga_push_batch(e, NULL, NULL, 0, NULL) == 0);
    EXPECT(ga_num_arrivals(e) == 0);
    EXPECT(ga_push(e, 3, fake) == GA_ERR_ARG && ga_push(e, 0, (float*)((size_t)fake + 4)) == GA_ERR_ARG);
    EXPECT(ga_set_option(e, 99, 1.0) == GA_ERR_ARG && ga_set_option(e, GA_OPT_WINDOW, 17.0) == GA_ERR_ARG);
    EXPECT(ga_get_stats(e, &s, &m) == GA_ERR_STATE);
    size_t need = ga_export_state(e, NULL, 0);
    EXPECT(need > 0);
    char* blob = (char*)malloc(need);
    EXPECT(blob && ga_export_state(e, blob, need) == need);
    EXPECT(ga_import_state(e, blob, need - 1) == GA_ERR_ARG);
    EXPECT(ga_import_state(e, blob, need) == GA_OK);
    blob[0] ^= 1;
    EXPECT(ga_import_state(e, blob, need) == GA_ERR_ARG);
    free(blob);
    ga_destroy(e);
    printf("sanitize api driver ok\n");
    return 0;
}
