// Device entry points of the synthetic-input generator (definitions in wl_gen.h). They fill
// whole vectors in device memory; values are bit-identical to wl_cpu.c at the same indices.
// Input generation only: nothing of the master's update rule lives here.
#include <cuda_runtime.h>

#include "wl_gen.h"

namespace {

// Element t of the local buffers is global element j0 + t (a rank may hold a sub-range).
__global__ void init_kernel(uint64_t seed, int64_t j0, int64_t n, float* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += stride)
        out[t] = wl_init(seed, j0 + t);
}

__global__ void grad_kernel(wl_spec sp, const int64_t* __restrict__ seg_off,
                            const float* __restrict__ seg_sigma, uint64_t noise_key,
                            uint64_t row_key, int64_t j0, int64_t n,
                            const float* __restrict__ sent, float* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += stride) {
        const int64_t j = j0 + t;
        const float sigma = seg_sigma[wl_segment(seg_off, sp.n_seg, j)];
        const float s = sp.quad ? sent[t] : 0.0f;
        out[t] = wl_grad_elem(&sp, noise_key, row_key, sigma, j, s);
    }
}

int grid_for(int64_t n) {
    int64_t g = (n + 255) / 256;
    const int64_t cap = 148 * 16;
    return (int)(g < cap ? (g > 0 ? g : 1) : cap);
}

}  // namespace

extern "C" {

int wl_cuda_init(uint64_t seed, int64_t j0, int64_t n, float* out_dev, void* stream) {
    init_kernel<<<grid_for(n), 256, 0, (cudaStream_t)stream>>>(seed, j0, n, out_dev);
    return (int)cudaGetLastError();
}

// Gradient of arrival k for global elements [j0, j0+n) from the parameters sent to the worker
// (sent_dev and out_dev hold that range only).
int wl_cuda_grad(const wl_spec* sp, const int64_t* seg_off_dev, const float* seg_sigma_dev,
                 int64_t k, int64_t j0, int64_t n, const float* sent_dev, float* out_dev,
                 void* stream) {
    const uint64_t noise_key = wl_key(sp->seed, WL_NOISE, (uint64_t)k);
    const uint64_t row_key = wl_key(sp->seed, WL_ROW, (uint64_t)k);
    if (j0 < 0 || n < 0 || j0 + n > sp->d) return (int)cudaErrorInvalidValue;
    if (n == 0) return 0;
    grad_kernel<<<grid_for(n), 256, 0, (cudaStream_t)stream>>>(
        *sp, seg_off_dev, seg_sigma_dev, noise_key, row_key, j0, n, sent_dev, out_dev);
    return (int)cudaGetLastError();
}

}  // extern "C"
