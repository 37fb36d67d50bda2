// Device entry points of the synthetic-input generator (definitions in wl_gen.h). They fill
// whole vectors in device memory; values are bit-identical to wl_cpu.c at the same indices.
// Input generation only: nothing of the master's update rule lives here.
#include <cuda_runtime.h>

#include "wl_gen.h"

namespace {

__global__ void init_kernel(uint64_t seed, int64_t d, float* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += stride)
        out[j] = wl_init(seed, j);
}

__global__ void grad_kernel(wl_spec sp, const int64_t* __restrict__ seg_off,
                            const float* __restrict__ seg_sigma, uint64_t noise_key,
                            uint64_t row_key, const float* __restrict__ sent,
                            float* __restrict__ out) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < sp.d; j += stride) {
        const float sigma = seg_sigma[wl_segment(seg_off, sp.n_seg, j)];
        const float s = sp.quad ? sent[j] : 0.0f;
        out[j] = wl_grad_elem(&sp, noise_key, row_key, sigma, j, s);
    }
}

int grid_for(int64_t n) {
    int64_t g = (n + 255) / 256;
    const int64_t cap = 148 * 16;
    return (int)(g < cap ? (g > 0 ? g : 1) : cap);
}

}  // namespace

extern "C" {

int wl_cuda_init(uint64_t seed, int64_t d, float* out_dev, void* stream) {
    init_kernel<<<grid_for(d), 256, 0, (cudaStream_t)stream>>>(seed, d, out_dev);
    return (int)cudaGetLastError();
}

// Gradient of arrival k for all d elements from the parameters sent to the worker.
int wl_cuda_grad(const wl_spec* sp, const int64_t* seg_off_dev, const float* seg_sigma_dev,
                 int64_t k, const float* sent_dev, float* out_dev, void* stream) {
    const uint64_t noise_key = wl_key(sp->seed, WL_NOISE, (uint64_t)k);
    const uint64_t row_key = wl_key(sp->seed, WL_ROW, (uint64_t)k);
    grad_kernel<<<grid_for(sp->d), 256, 0, (cudaStream_t)stream>>>(
        *sp, seg_off_dev, seg_sigma_dev, noise_key, row_key, sent_dev, out_dev);
    return (int)cudaGetLastError();
}

}  // extern "C"
