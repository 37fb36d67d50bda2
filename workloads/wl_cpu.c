/* CPU side of the seeded synthetic inputs (initial parameters, curvature, target, stand-in worker
 * gradient). It feeds the CPU oracle's runs. Input generation only: nothing of the master's
 * update rule lives here.
 *
 * This file is a self-contained implementation written from the definitions below; it shares no
 * source with the device generator (wl_gen.h / wl_cuda.cu), so that the test comparing the two
 * bit for bit compares two programs, not one file with itself.
 *
 * Definitions (all integer arithmetic modulo 2^64):
 *   finalise(z): z ^= z >> 30; z *= 0xBF58476D1CE4E5B9; z ^= z >> 27; z *= 0x94D049BB133111EB;
 *                z ^= z >> 31                              (output function of SplitMix64)
 *   PHI = 0x9E3779B97F4A7C15
 *   stream(seed, tag, a) = finalise(finalise(seed + PHI*(tag+1)) + a)
 *   draw(stream, b)      = finalise(stream + PHI*(b+1))    (output number b of SplitMix64 seeded with `stream`)
 *   uniform in (0,1):  ((draw >> 41) + 1/2) / 2^23
 *   unit-variance noise: (sum of the four 16-bit fields of a draw - 131070) * sqrt(3)/65536
 *   curvature a_j = 1/2 + 3/2 u(stream(seed,1,0), j); target theta*_j = noise(stream(seed,2,0), j) / 10;
 *   start theta0_j = noise(stream(seed,3,0), j) / 20   (as products with the fp32 constants 0.1f, 0.05f)
 *   gradient of arrival k at element j from the parameters sent (s_j), sigma = noise scale of j's segment:
 *       g_j = a_j * (s_j - theta*_j) + sigma * noise(stream(seed,0,k), j)     (fused multiply-add)
 *     without the quadratic term when quad == 0; elements below emb_elems form rows of emb_row
 *     elements and a row r contributes only if draw(stream(seed,4,k), r) < row_thresh, else g = 0.
 * Every fp32 operation is rounded once (build with -ffp-contract=off; the one fused operation is
 * written as fmaf).
 *
 * Entry points take arrays of GLOBAL element indices (idx == NULL: the dense range [0, n)), so a
 * sampled subset of a large vector gets exactly the values the full vector would. */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

enum stream_tag { TAG_NOISE = 0, TAG_CURVATURE = 1, TAG_TARGET = 2, TAG_START = 3, TAG_ROW = 4 };

static const uint64_t PHI = 0x9E3779B97F4A7C15ULL;

static uint64_t finalise(uint64_t z) {
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

static uint64_t stream(uint64_t seed, uint64_t tag, uint64_t a) {
    const uint64_t first = finalise(seed + PHI * (tag + 1));
    return finalise(first + a);
}

static uint64_t draw(uint64_t strm, uint64_t b) { return finalise(strm + PHI * (b + 1)); }

/* top 23 bits + 1/2, scaled by 2^-23: a 24-bit odd integer times 2^-24, exact in fp32 */
static float uniform_open(uint64_t w) {
    const uint32_t top = (uint32_t)(w >> 41);
    return ldexpf((float)(2u * top + 1u), -24);
}

static float noise_unit(uint64_t w) {
    int sum = 0;
    for (int field = 0; field < 4; ++field) sum += (int)((w >> (16 * field)) & 0xFFFFu);
    const float scale = (float)(1.7320508075688772 / 65536.0);   /* sqrt(3) / 2^16, rounded to fp32 */
    return (float)(sum - 131070) * scale;
}

/* layout shared with the Python side (ctypes) */
typedef struct {
    uint64_t seed;
    int64_t d;
    int32_t quad;
    int32_t n_seg;
    int64_t emb_elems;
    int64_t emb_row;
    uint64_t row_thresh;
} workload_spec;

static int64_t element(const int64_t* idx, int64_t t) { return idx ? idx[t] : t; }

/* number of segment starts <= j, minus one: the segment that holds j */
static int segment_of(const int64_t* seg_off, int n_seg, int64_t j) {
    int first = 1, count = n_seg - 1;          /* search seg_off[1 .. n_seg-1] for the first start > j */
    while (count > 0) {
        const int half = count / 2;
        if (seg_off[first + half] <= j) { first += half + 1; count -= half + 1; }
        else count = half;
    }
    return first - 1;
}

uint64_t wl_cpu_mix64(uint64_t z) { return finalise(z); }
uint64_t wl_cpu_hash(uint64_t seed, uint64_t tag, uint64_t a, uint64_t b) { return draw(stream(seed, tag, a), b); }
float wl_cpu_uniform(uint64_t w) { return uniform_open(w); }
float wl_cpu_xi(uint64_t w) { return noise_unit(w); }

void wl_cpu_init(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    const uint64_t strm = stream(seed, TAG_START, 0);
    for (int64_t t = 0; t < n; ++t) out[t] = 0.05f * noise_unit(draw(strm, (uint64_t)element(idx, t)));
}

void wl_cpu_target(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    const uint64_t strm = stream(seed, TAG_TARGET, 0);
    for (int64_t t = 0; t < n; ++t) out[t] = 0.1f * noise_unit(draw(strm, (uint64_t)element(idx, t)));
}

void wl_cpu_curv(uint64_t seed, const int64_t* idx, int64_t n, float* out) {
    const uint64_t strm = stream(seed, TAG_CURVATURE, 0);
    for (int64_t t = 0; t < n; ++t) out[t] = fmaf(1.5f, uniform_open(draw(strm, (uint64_t)element(idx, t))), 0.5f);
}

/* Gradient of arrival k at the listed elements, from the parameters the worker was sent
 * (sent[t] belongs to element idx[t]). */
void wl_cpu_grad(const workload_spec* sp, const int64_t* seg_off, const float* seg_sigma, int64_t k,
                 const int64_t* idx, int64_t n, const float* sent, float* out) {
    const uint64_t noise_stream = stream(sp->seed, TAG_NOISE, (uint64_t)k);
    const uint64_t row_stream = stream(sp->seed, TAG_ROW, (uint64_t)k);
    const uint64_t curv_stream = stream(sp->seed, TAG_CURVATURE, 0);
    const uint64_t target_stream = stream(sp->seed, TAG_TARGET, 0);
    for (int64_t t = 0; t < n; ++t) {
        const int64_t j = element(idx, t);
        if (j < sp->emb_elems) {                       /* sparse region: whole rows switch on and off */
            const uint64_t row = (uint64_t)(j / sp->emb_row);
            if (draw(row_stream, row) >= sp->row_thresh) { out[t] = 0.0f; continue; }
        }
        const float sigma = seg_sigma[segment_of(seg_off, sp->n_seg, j)];
        const float noise = sigma * noise_unit(draw(noise_stream, (uint64_t)j));
        if (!sp->quad) { out[t] = noise; continue; }
        const float a = fmaf(1.5f, uniform_open(draw(curv_stream, (uint64_t)j)), 0.5f);
        const float target = 0.1f * noise_unit(draw(target_stream, (uint64_t)j));
        out[t] = fmaf(a, sent[t] - target, noise);
    }
}
