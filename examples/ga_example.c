/* Minimal use of the C ABI from plain C (no Python, no torch): one master, two workers,
 * Gap-Aware variant, a constant gradient. Build:
 *   gcc -I include examples/ga_example.c -o ga_example \
 *       -L paper_1909_10802_b200 -lga -L/usr/local/cuda/lib64 -lcudart -Wl,-rpath,$PWD/paper_1909_10802_b200
 * Prints theta[0] after each arrival and the delays; exits non-zero on any error. */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>

#include "ga.h"

#define CHECK(x)                                                        \
    do {                                                                \
        if ((x) < 0) {                                                  \
            fprintf(stderr, "%s failed: %s\n", #x, ga_last_error());   \
            return 1;                                                   \
        }                                                               \
    } while (0)

int main(void) {
    const size_t d = 1000;
    float host[1000];
    float *theta0 = NULL, *grad = NULL, *out = NULL;
    if (cudaMalloc((void**)&theta0, d * sizeof(float)) != cudaSuccess ||
        cudaMalloc((void**)&grad, d * sizeof(float)) != cudaSuccess ||
        cudaMalloc((void**)&out, d * sizeof(float)) != cudaSuccess) {
        fprintf(stderr, "no CUDA device\n");
        return 2;
    }
    for (size_t j = 0; j < d; ++j) host[j] = 1.0f;
    cudaMemcpy(theta0, host, sizeof host, cudaMemcpyHostToDevice);
    for (size_t j = 0; j < d; ++j) host[j] = 0.5f;
    cudaMemcpy(grad, host, sizeof host, cudaMemcpyHostToDevice);

    ga_engine* e = ga_create(d, 2, 0.1f, 0.0f, 0.999f, GA_GA);
    if (!e) {
        fprintf(stderr, "ga_create: %s\n", ga_last_error());
        return 1;
    }
    CHECK(ga_set_params(e, theta0));
    /* worker 1 pushes three times (pulling after each), then worker 0, still holding theta_0, pushes */
    const int schedule[4] = {1, 1, 1, 0};
    const float* grads[4] = {grad, grad, grad, grad};
    int64_t delays[4];
    CHECK(ga_push_batch(e, schedule, grads, 4, delays));
    CHECK(ga_get(e, GA_THETA, out));
    cudaMemcpy(host, out, sizeof host, cudaMemcpyDeviceToHost);
    /* three unpenalised steps of 0.05, then one divided by a Gap of (about) 4 */
    printf("delays %lld %lld %lld %lld theta %.6f\n", (long long)delays[0], (long long)delays[1],
           (long long)delays[2], (long long)delays[3], host[0]);
    ga_destroy(e);
    cudaFree(theta0);
    cudaFree(grad);
    cudaFree(out);
    return 0;
}
