/* What one ga_push_batch call costs from plain C when the vector is small enough to live in the
 * L2 cache (272,474 parameters -- a CIFAR ResNet-20 -- 8 workers): 10,000 calls of one fused
 * window of 8 arrivals each, no Python in the loop. Prints the host time per call while calls
 * are only being enqueued, and the time per call once the GPU has finished them all, i.e. the
 * sustained rate at which a master can take windows. Build:
 *   gcc -O2 -I include examples/ga_call_timing.c -o ga_call_timing \
 *       -L paper_1909_10802_b200 -lga -L/usr/local/cuda/lib64 -lcudart -Wl,-rpath,$PWD/paper_1909_10802_b200
 * Usage: ga_call_timing [n_params [n_workers [calls]]] */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>
#include <time.h>

#include "ga.h"

static double now(void) {
    struct timespec t;
    clock_gettime(CLOCK_MONOTONIC, &t);
    return (double)t.tv_sec + 1e-9 * (double)t.tv_nsec;
}

int main(int argc, char** argv) {
    const size_t d = argc > 1 ? (size_t)atoll(argv[1]) : 272474;
    const int n = argc > 2 ? atoi(argv[2]) : 8;
    const int calls = argc > 3 ? atoi(argv[3]) : 10000;
    if (n < 1 || n > GA_MAX_WINDOW || d == 0 || calls < 1) { fprintf(stderr, "bad arguments\n"); return 2; }
    float* host = (float*)malloc(d * sizeof(float));
    float* theta0 = NULL;
    float* grads[GA_MAX_WINDOW];
    if (!host || cudaMalloc((void**)&theta0, d * sizeof(float)) != cudaSuccess) { fprintf(stderr, "no CUDA device\n"); return 2; }
    for (size_t j = 0; j < d; ++j) host[j] = 0.05f * (float)((j * 2654435761u) % 2001 - 1000) / 1000.0f;
    cudaMemcpy(theta0, host, d * sizeof(float), cudaMemcpyHostToDevice);
    int schedule[GA_MAX_WINDOW];
    const float* grad_ptrs[GA_MAX_WINDOW];
    for (int i = 0; i < n; ++i) {      /* one fixed, small gradient per worker */
        if (cudaMalloc((void**)&grads[i], d * sizeof(float)) != cudaSuccess) return 2;
        for (size_t j = 0; j < d; ++j) host[j] = 1e-3f * (float)(((j + 17u * i) * 2246822519u) % 2001 - 1000) / 1000.0f;
        cudaMemcpy(grads[i], host, d * sizeof(float), cudaMemcpyHostToDevice);
        schedule[i] = i;
        grad_ptrs[i] = grads[i];
    }
    ga_engine* e = ga_create(d, n, 0.1f, 0.9f, 0.999f, GA_GA);
    if (!e || ga_set_params(e, theta0) < 0) { fprintf(stderr, "%s\n", ga_last_error()); return 1; }
    for (int c = 0; c < 100; ++c)      /* warm-up */
        if (ga_push_batch(e, schedule, grad_ptrs, n, NULL) < 0) { fprintf(stderr, "%s\n", ga_last_error()); return 1; }
    cudaDeviceSynchronize();
    const double t0 = now();
    for (int c = 0; c < calls; ++c)
        if (ga_push_batch(e, schedule, grad_ptrs, n, NULL) < 0) { fprintf(stderr, "%s\n", ga_last_error()); return 1; }
    const double t1 = now();
    cudaDeviceSynchronize();
    const double t2 = now();
    printf("params %zu workers %d calls %d arrivals_per_call %d enqueue_us_per_call %.2f total_us_per_call %.2f "
           "param_updates_per_s %.3e\n", d, n, calls, n, 1e6 * (t1 - t0) / calls, 1e6 * (t2 - t0) / calls,
           (double)d * n * calls / (t2 - t0));
    ga_destroy(e);
    for (int i = 0; i < n; ++i) cudaFree(grads[i]);
    cudaFree(theta0);
    free(host);
    return 0;
}
