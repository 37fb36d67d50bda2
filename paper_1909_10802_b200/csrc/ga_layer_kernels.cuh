// Layer-wise (and, with one layer, global) Gap-Aware master for sm_100a.
//
// Section 5.3 of the paper: G_p = ||theta_p - theta^i_p|| / C_p + 1, one number per layer, and the
// gradient of layer p is multiplied by 1/G_p before the momentum step. The norm is a reduction
// over the layer, so one arrival takes two passes over the vector:
//   1. ga_layer_dist_kernel    per-tile partial sums of (theta - theta^i)^2          (8 B/param)
//      ga_layer_gap_kernel     per layer: sum the partials, form C_p, G_p, 1/G_p
//   2. ga_layer_update_kernel  v <- gamma v + g/G_p ; theta <- theta - eta v ; save theta;
//                              per-tile partial sums of v^2                           (24 B/param)
//      ga_layer_refresh_kernel per layer: m_p <- beta m_p + (1-beta) ||v_p||^2
// A tile is at most kLayerTile consecutive elements of ONE layer (the host cuts the layers into
// tiles), so a block never mixes layers. Squared norms are accumulated in fp64 in a fixed order
// (thread-strided, warp shuffles, warps in order; tiles of a layer in order) and rounded to fp32
// once, which makes the result reproducible run to run.
#pragma once

#include <cuda_runtime.h>

#include "ga_kernels.cuh"

namespace ga {

constexpr int kLayerTile = 4096;
constexpr int kLayerThreads = 256;

struct Tile {
    long long start;  // first element
    int len;          // 1..kLayerTile
    int layer;
};

// Sum over the block in a fixed order; the result is valid in thread 0.
__device__ __forceinline__ double block_sum(double x) {
    __shared__ double s_part[kLayerThreads / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = x;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < kLayerThreads / 32; ++w) total += s_part[w];
    return total;
}

// Element range of a tile split into an unaligned head, a 128-bit aligned body and a tail.
struct TileRange {
    long long b, ab, ae, e;
    __device__ explicit TileRange(const Tile& t) {
        b = t.start;
        e = b + t.len;
        ab = (b + 3) & ~3LL;
        if (ab > e) ab = e;
        ae = e & ~3LL;
        if (ae < ab) ae = ab;
    }
};

__global__ void __launch_bounds__(kLayerThreads)
ga_layer_dist_kernel(const float* __restrict__ theta, const float* __restrict__ saved,
                     const Tile* __restrict__ tiles, double* __restrict__ partial) {
    const TileRange r(tiles[blockIdx.x]);
    double acc = 0.0;
    auto one = [&](float t, float s) {
        const float diff = __fsub_rn(t, s);
        acc += (double)diff * (double)diff;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) one(theta[i], saved[i]);
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        const float4 t = *reinterpret_cast<const float4*>(theta + 4 * q);
        const float4 s = ld_stream(saved + 4 * q);
        one(t.x, s.x); one(t.y, s.y); one(t.z, s.z); one(t.w, s.w);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) one(theta[i], saved[i]);
    const double total = block_sum(acc);
    if (threadIdx.x == 0) partial[blockIdx.x] = total;
}

// Sum of the partials of layer p (block p), in a fixed order; valid in thread 0.
__device__ __forceinline__ double layer_total(const double* __restrict__ partial, const int* __restrict__ tile_begin) {
    const int lo = tile_begin[blockIdx.x], hi = tile_begin[blockIdx.x + 1];
    double acc = 0.0;
    for (int q = lo + threadIdx.x; q < hi; q += kLayerThreads) acc += partial[q];
    return block_sum(acc);
}

__global__ void __launch_bounds__(kLayerThreads)
ga_layer_gap_kernel(const double* __restrict__ partial, const int* __restrict__ tile_begin,
                    const float* __restrict__ m_layer, float inv_bias, Hyper h,
                    float* __restrict__ gap, float* __restrict__ inv_gap) {
    const double total = layer_total(partial, tile_begin);
    if (threadIdx.x == 0) {
        const float dist = (float)sqrt(total);
        const float C = __fmul_rn(h.eta_max, __fadd_rn(__fsqrt_rn(__fmul_rn(m_layer[blockIdx.x], inv_bias)), h.eps));
        const float G = __fadd_rn(__fdiv_rn(dist, C), 1.0f);
        gap[blockIdx.x] = G;
        inv_gap[blockIdx.x] = __frcp_rn(G);
    }
}

__global__ void __launch_bounds__(kLayerThreads)
ga_layer_update_kernel(float* __restrict__ theta, float* __restrict__ vel, const float* __restrict__ grad,
                       float* __restrict__ saved, int write_saved, const Tile* __restrict__ tiles,
                       const float* __restrict__ inv_gap, float eta, Hyper h, double* __restrict__ partial) {
    const Tile t = tiles[blockIdx.x];
    const TileRange r(t);
    const float inv = inv_gap[t.layer];
    double acc = 0.0;
    auto one = [&](float& th, float& v, float g) {
        if (h.wd != 0.0f) g = __fmaf_rn(h.wd, th, g);      // decay element: part of the gradient
        v = __fmaf_rn(h.gamma, v, __fmul_rn(inv, g));      // (1/G_p) g, then the momentum step
        if (h.nesterov) th = __fmaf_rn(-eta, __fmaf_rn(h.gamma, v, __fmul_rn(inv, g)), th);
        else th = __fmaf_rn(-eta, v, th);
        acc += (double)v * (double)v;
    };
    auto scalar = [&](long long i) {
        float th = theta[i], v = vel[i];
        one(th, v, grad[i]);
        theta[i] = th;
        vel[i] = v;
        if (write_saved) saved[i] = th;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) scalar(i);
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        float4 th = *reinterpret_cast<const float4*>(theta + 4 * q);
        float4 v = *reinterpret_cast<const float4*>(vel + 4 * q);
        const float4 g = ld_stream(grad + 4 * q);
        one(th.x, v.x, g.x); one(th.y, v.y, g.y); one(th.z, v.z, g.z); one(th.w, v.w, g.w);
        *reinterpret_cast<float4*>(theta + 4 * q) = th;
        *reinterpret_cast<float4*>(vel + 4 * q) = v;
        if (write_saved) st_stream(saved + 4 * q, th);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) scalar(i);
    const double total = block_sum(acc);
    if (threadIdx.x == 0) partial[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kLayerThreads)
ga_layer_refresh_kernel(const double* __restrict__ partial, const int* __restrict__ tile_begin,
                        float* __restrict__ m_layer, Hyper h) {
    const double total = layer_total(partial, tile_begin);
    if (threadIdx.x == 0)
        m_layer[blockIdx.x] = __fmaf_rn(h.beta, m_layer[blockIdx.x], __fmul_rn(h.one_minus_beta, (float)total));
}

}  // namespace ga
