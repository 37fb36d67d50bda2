// Layer-wise (and, with one layer, global) Gap-Aware master for sm_100a.
//
// Section 5.3 of the paper: G_p = ||theta_p - theta^i_p|| / C_p + 1, one number per layer, and the
// gradient of layer p is multiplied by 1/G_p before the momentum step. The norm is a reduction
// over the layer and must be known before the layer's update, so arrivals cannot be fused in
// time the way the parameter-wise kernel fuses them. What can be fused is the NEXT arrival's
// norm: inside one ga_push_batch call the next arriving worker is known, so the pass that
// applies arrival j also accumulates ||theta_new - theta^{next}||^2 while theta_new is in
// registers. One call of K arrivals is therefore
//   ga_layer_dist_kernel    once, for the first arrival: ||theta - theta^i||^2 per layer     (8 B/param)
//   ga_layer_update_kernel  K times: v <- gamma v + g/G_p ; theta <- theta - eta v ; save theta ;
//                           ||v_p||^2 ; and, for the next arrival, ||theta - theta^next||^2  (28 B/param)
// A tile is at most kLayerTile consecutive elements of ONE layer (the host cuts the layers into
// tiles), so a block never mixes layers. Each block leaves its tile's partial sums in global
// memory and takes a ticket of its layer; the block that draws a layer's last ticket sums the
// layer's partials and does the per-layer step (refresh of m_p, then C_p, G_p and 1/G_p of the
// next arrival) -- one ticket counter per layer, so the layers finish independently. Squared norms
// are accumulated in fp64 in a fixed order (thread-strided over the tile, warp shuffles, warps in
// order; tiles of a layer thread-strided in index order) and rounded to fp32 once, which makes
// the result independent of which block happens to come last, and reproducible run to run.
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

// Per-layer tables of the engine (device memory).
struct LayerTables {
    const Tile* tiles;
    const int* tile_begin;   // n_layers + 1: tiles of layer p are [tile_begin[p], tile_begin[p+1])
    double* partial_v;       // per tile: sum of v^2 after the update
    double* partial_d;       // per tile: sum of (theta - saved copy)^2
    unsigned int* ticket;    // per layer, 0 between launches
    float* m_layer;          // m_p of the C algorithm
    float* gap;              // G_p of the most recent arrival
    float* inv_gap;          // 1 / G_p of the arrival about to be applied
};

// Sums of two values over the block in a fixed order; valid in thread 0.
__device__ __forceinline__ void block_sum2(double& x, double& y) {
    __shared__ double s_x[kLayerThreads / 32], s_y[kLayerThreads / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        x += __shfl_xor_sync(0xffffffffu, x, o);
        y += __shfl_xor_sync(0xffffffffu, y, o);
    }
    __syncthreads();                     // the arrays may still be read from an earlier call
    if ((threadIdx.x & 31) == 0) { s_x[threadIdx.x >> 5] = x; s_y[threadIdx.x >> 5] = y; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tx = 0.0, ty = 0.0;
        for (int w = 0; w < kLayerThreads / 32; ++w) { tx += s_x[w]; ty += s_y[w]; }
        x = tx;
        y = ty;
    }
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

// Thread 0 has just written this tile's partial sums. Returns true (to every thread) in the block
// that is the last of its layer to get here; that block then sees all partials of the layer.
__device__ __forceinline__ bool last_tile_of_layer(const LayerTables& T, int layer) {
    __shared__ int s_last;
    if (threadIdx.x == 0) {
        __threadfence();                                     // partials before the ticket
        const unsigned int n = (unsigned int)(T.tile_begin[layer + 1] - T.tile_begin[layer]);
        const unsigned int got = atomicAdd(&T.ticket[layer], 1u);
        s_last = (got == n - 1);
        if (s_last) { T.ticket[layer] = 0; __threadfence(); }   // ready for the next launch; see all partials
    }
    __syncthreads();
    return s_last != 0;
}

// Sums of a layer's partials (both arrays) in index order; valid in thread 0.
__device__ __forceinline__ void layer_totals(const LayerTables& T, int layer, bool want_v, bool want_d, double& tv,
                                             double& td) {
    const int lo = T.tile_begin[layer], hi = T.tile_begin[layer + 1];
    tv = 0.0;
    td = 0.0;
    for (int q = lo + threadIdx.x; q < hi; q += kLayerThreads) {
        if (want_v) tv += __ldcg(T.partial_v + q);
        if (want_d) td += __ldcg(T.partial_d + q);
    }
    block_sum2(tv, td);
}

// C_p, G_p and 1/G_p of a layer from its squared distance (thread 0 of the layer's last block).
__device__ __forceinline__ void layer_gap(const LayerTables& T, int layer, double dist2, float m_p, float inv_bias,
                                          const Hyper& h) {
    const float dist = (float)sqrt(dist2);
    const float C = __fmul_rn(h.eta_max, __fadd_rn(__fsqrt_rn(__fmul_rn(m_p, inv_bias)), h.eps));
    const float G = __fadd_rn(__fdiv_rn(dist, C), 1.0f);
    T.gap[layer] = G;
    T.inv_gap[layer] = __frcp_rn(G);
}

// First arrival of a call: ||theta_p - theta^i_p||^2 per layer, then its Gap.
__global__ void __launch_bounds__(kLayerThreads)
ga_layer_dist_kernel(const float* __restrict__ theta, const float* __restrict__ saved, LayerTables T,
                     float inv_bias, Hyper h) {
    const Tile t = T.tiles[blockIdx.x];
    const TileRange r(t);
    double acc = 0.0, none = 0.0;
    auto one = [&](float th, float s) {
        const float diff = __fsub_rn(th, s);
        acc += (double)diff * (double)diff;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) one(theta[i], saved[i]);
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        const float4 th = *reinterpret_cast<const float4*>(theta + 4 * q);
        const float4 s = ld_stream(saved + 4 * q);
        one(th.x, s.x); one(th.y, s.y); one(th.z, s.z); one(th.w, s.w);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) one(theta[i], saved[i]);
    block_sum2(acc, none);
    if (threadIdx.x == 0) T.partial_d[blockIdx.x] = acc;
    if (!last_tile_of_layer(T, t.layer)) return;
    double tv, td;
    layer_totals(T, t.layer, false, true, tv, td);
    if (threadIdx.x == 0) layer_gap(T, t.layer, td, T.m_layer[t.layer], inv_bias, h);
}

// One arrival. next_mode: 0 = the next arrival is not known (last of the call); 1 = its worker's saved
// copy is `next`; 2 = the same worker arrives again, whose copy is the theta being saved right now,
// so its distance is exactly 0. inv_bias_next is 1/(1-beta^k') for the C of the next arrival.
__global__ void __launch_bounds__(kLayerThreads)
ga_layer_update_kernel(float* __restrict__ theta, float* __restrict__ vel, const float* __restrict__ grad,
                       float* __restrict__ saved, int write_saved, const float* __restrict__ next, int next_mode,
                       LayerTables T, float eta, Hyper h, float inv_bias_next) {
    const Tile t = T.tiles[blockIdx.x];
    const TileRange r(t);
    const float inv = T.inv_gap[t.layer];
    const bool look = next_mode == 1;
    double acc_v = 0.0, acc_d = 0.0;
    auto one = [&](float& th, float& v, float g, float s_next) {
        if (h.wd != 0.0f) g = __fmaf_rn(h.wd, th, g);      // decay element: part of the gradient
        v = __fmaf_rn(h.gamma, v, __fmul_rn(inv, g));      // (1/G_p) g, then the momentum step
        if (h.nesterov) th = __fmaf_rn(-eta, __fmaf_rn(h.gamma, v, __fmul_rn(inv, g)), th);
        else th = __fmaf_rn(-eta, v, th);
        acc_v += (double)v * (double)v;
        if (look) {
            const float diff = __fsub_rn(th, s_next);
            acc_d += (double)diff * (double)diff;
        }
    };
    auto scalar = [&](long long i) {
        float th = theta[i], v = vel[i];
        one(th, v, grad[i], look ? next[i] : 0.f);
        theta[i] = th;
        vel[i] = v;
        if (write_saved) saved[i] = th;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) scalar(i);
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        float4 th = *reinterpret_cast<const float4*>(theta + 4 * q);
        float4 v = *reinterpret_cast<const float4*>(vel + 4 * q);
        const float4 g = ld_stream(grad + 4 * q);
        const float4 s = look ? ld_stream(next + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
        one(th.x, v.x, g.x, s.x); one(th.y, v.y, g.y, s.y); one(th.z, v.z, g.z, s.z); one(th.w, v.w, g.w, s.w);
        *reinterpret_cast<float4*>(theta + 4 * q) = th;
        *reinterpret_cast<float4*>(vel + 4 * q) = v;
        if (write_saved) st_stream(saved + 4 * q, th);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) scalar(i);
    block_sum2(acc_v, acc_d);
    if (threadIdx.x == 0) {
        T.partial_v[blockIdx.x] = acc_v;
        T.partial_d[blockIdx.x] = acc_d;
    }
    if (!last_tile_of_layer(T, t.layer)) return;
    double tv, td;
    layer_totals(T, t.layer, true, look, tv, td);
    if (threadIdx.x == 0) {
        const float m_new = __fmaf_rn(h.beta, T.m_layer[t.layer], __fmul_rn(h.one_minus_beta, (float)tv));
        T.m_layer[t.layer] = m_new;
        if (next_mode != 0) layer_gap(T, t.layer, td, m_new, inv_bias_next, h);   // mode 2: td = 0
    }
}

}  // namespace ga
