/* Seeded synthetic inputs for the parameter-server update: initial parameters, the
 * stand-in "worker" gradient and the per-segment noise scales. Input generation only:
 * nothing of the master's update rule lives here. This header is the DEVICE generator
 * (compiled by nvcc into wl_cuda.cu); the CPU side that feeds the oracle is a separate program,
 * wl_cpu.c, written from the same definitions and sharing no source with this file. A GPU test
 * holds the two to bit-identical outputs.
 *
 * Every random quantity is a pure function of (seed, stream tag, a, b):
 *
 *   mix64(z):  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9
 *              z = (z ^ (z >> 27)) * 0x94D049BB133111EB
 *              return z ^ (z >> 31)                      (the SplitMix64 output function)
 *   GOLD    =  0x9E3779B97F4A7C15
 *   key(seed, tag, a) = mix64( mix64(seed + GOLD*(tag+1)) + a )
 *   word(key, b)      = mix64( key + GOLD*(b+1) )        (output b of SplitMix64 seeded with key)
 *
 *   uniform u in (0,1): ((word >> 41) + 0.5) * 2^-23                    (exact in fp32)
 *   noise xi, unit variance: the four 16-bit fields of one word are summed (exact integer),
 *              centred by 131070 and scaled by sqrt(3)/65536 (one fp32 multiply)
 *
 * Gradient of the quadratic stand-in loss for arrival k (1-based), element j, computed from
 * the parameters the worker was sent (s_j):
 *   g_j = fma(a_j, s_j - theta*_j, sigma_l(j) * xi(seed, NOISE, k, j))
 *   a_j = fma(1.5, u(seed, CURV, 0, j), 0.5)        in [0.5, 2]
 *   theta*_j = 0.1 * xi(seed, TARGET, 0, j)
 *   theta0_j = 0.05 * xi(seed, INIT, 0, j)
 * With quad == 0 the a_j term is absent (g = sigma * xi). Elements j < emb_elems form rows of
 * emb_row elements; row r is active for arrival k iff word(key(seed, ROW, k), r) < row_thresh,
 * and an inactive row's gradient is exactly 0.
 * Each operation is a single IEEE fp32 operation (no contraction) on both compilers.
 */
#ifndef WL_GEN_H
#define WL_GEN_H

#include <stdint.h>

#ifdef __CUDACC__
#define WL_HD __host__ __device__ __forceinline__
#else
#define WL_HD static inline
#include <math.h>
#endif

enum { WL_NOISE = 0, WL_CURV = 1, WL_TARGET = 2, WL_INIT = 3, WL_ROW = 4, WL_SIGMA = 5,
       WL_TIME = 6, WL_SPEED = 7 };

#define WL_GOLD 0x9E3779B97F4A7C15ULL

WL_HD uint64_t wl_mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

WL_HD uint64_t wl_key(uint64_t seed, uint64_t tag, uint64_t a) {
    return wl_mix64(wl_mix64(seed + WL_GOLD * (tag + 1)) + a);
}

WL_HD uint64_t wl_word(uint64_t key, uint64_t b) { return wl_mix64(key + WL_GOLD * (b + 1)); }

/* single-rounded fp32 operations on either compiler */
#if defined(__CUDA_ARCH__)
#define WL_MUL(a, b) __fmul_rn((a), (b))
#define WL_SUB(a, b) __fsub_rn((a), (b))
#define WL_FMA(a, b, c) __fmaf_rn((a), (b), (c))
#else
#define WL_MUL(a, b) ((float)(a) * (float)(b))
#define WL_SUB(a, b) ((float)(a) - (float)(b))
#define WL_FMA(a, b, c) fmaf((a), (b), (c))
#endif

WL_HD float wl_uniform(uint64_t w) {
    /* ((w >> 41) + 0.5) * 2^-23 : a 24-bit integer times a power of two, exact */
    return (float)(2 * (int64_t)(w >> 41) + 1) * 0x1p-24f;
}

WL_HD float wl_xi(uint64_t w) {
    const int32_t s = (int32_t)(w & 0xFFFF) + (int32_t)((w >> 16) & 0xFFFF) +
                      (int32_t)((w >> 32) & 0xFFFF) + (int32_t)(w >> 48);
    return WL_MUL((float)(s - 131070), 0x1.bb67aep-16f); /* sqrt(3)/65536 rounded to fp32 */
}

typedef struct {
    uint64_t seed;
    int64_t d;            /* number of parameters */
    int32_t quad;         /* 1: g has the a*(s - theta*) term */
    int32_t n_seg;        /* number of layer segments */
    int64_t emb_elems;    /* elements [0, emb_elems) are rows of emb_row elements; 0 = none */
    int64_t emb_row;
    uint64_t row_thresh;  /* a row is active iff its word < row_thresh */
} wl_spec;

WL_HD float wl_curv(uint64_t seed, int64_t j) {
    return WL_FMA(1.5f, wl_uniform(wl_word(wl_key(seed, WL_CURV, 0), (uint64_t)j)), 0.5f);
}
WL_HD float wl_target(uint64_t seed, int64_t j) {
    return WL_MUL(0.1f, wl_xi(wl_word(wl_key(seed, WL_TARGET, 0), (uint64_t)j)));
}
WL_HD float wl_init(uint64_t seed, int64_t j) {
    return WL_MUL(0.05f, wl_xi(wl_word(wl_key(seed, WL_INIT, 0), (uint64_t)j)));
}

/* index of the segment holding element j: largest l with seg_off[l] <= j */
WL_HD int wl_segment(const int64_t* seg_off, int n_seg, int64_t j) {
    int lo = 0, hi = n_seg - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (seg_off[mid] <= j) lo = mid; else hi = mid - 1;
    }
    return lo;
}

/* noise_key = wl_key(seed, WL_NOISE, k), row_key = wl_key(seed, WL_ROW, k) */
WL_HD float wl_grad_elem(const wl_spec* sp, uint64_t noise_key, uint64_t row_key, float sigma,
                         int64_t j, float s_j) {
    if (j < sp->emb_elems) {
        const uint64_t r = (uint64_t)(j / sp->emb_row);
        if (wl_word(row_key, r) >= sp->row_thresh) return 0.0f;
    }
    const float noise = WL_MUL(sigma, wl_xi(wl_word(noise_key, (uint64_t)j)));
    if (!sp->quad) return noise;
    return WL_FMA(wl_curv(sp->seed, j), WL_SUB(s_j, wl_target(sp->seed, j)), noise);
}

#endif
