/* CPU entry points of the synthetic-input generator (see wl_gen.h for the definitions).
 * Each takes an array of GLOBAL element indices, so that a sampled subset of a large
 * parameter vector gets exactly the values the full vector would. idx == NULL means
 * the dense range [0, n). Build: gcc -O2 -ffp-contract=off -fPIC -shared. */
#include "wl_gen.h"

#include <stddef.h>

static int64_t at(const int64_t* idx, int64_t t) { return idx ? idx[t] : t; }

uint64_t wl_cpu_mix64(uint64_t z) { return wl_mix64(z); }
uint64_t wl_cpu_hash(uint64_t seed, uint64_t tag, uint64_t a, uint64_t b) {
    return wl_word(wl_key(seed, tag, a), b);
}
float wl_cpu_uniform(uint64_t w) { return wl_uniform(w); }
float wl_cpu_xi(uint64_t w) { return wl_xi(w); }

void wl_cpu_init(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    for (int64_t t = 0; t < n; ++t) out[t] = wl_init(seed, at(idx, t));
}
void wl_cpu_target(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    for (int64_t t = 0; t < n; ++t) out[t] = wl_target(seed, at(idx, t));
}
void wl_cpu_curv(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    for (int64_t t = 0; t < n; ++t) out[t] = wl_curv(seed, at(idx, t));
}

/* Gradient for arrival k at the listed elements, from the parameters the worker was sent
 * (sent[t] belongs to element idx[t]). */
void wl_cpu_grad(const wl_spec* sp, const int64_t* seg_off, const float* seg_sigma, int64_t k,
                 const int64_t* idx, int64_t n, const float* sent, float* out) {
    const uint64_t noise_key = wl_key(sp->seed, WL_NOISE, (uint64_t)k);
    const uint64_t row_key = wl_key(sp->seed, WL_ROW, (uint64_t)k);
    for (int64_t t = 0; t < n; ++t) {
        const int64_t j = at(idx, t);
        const float sigma = seg_sigma[wl_segment(seg_off, sp->n_seg, j)];
        out[t] = wl_grad_elem(sp, noise_key, row_key, sigma, j, sent[t]);
    }
}
