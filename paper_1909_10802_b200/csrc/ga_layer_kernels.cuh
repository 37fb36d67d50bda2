// Layer-wise (and, with one layer, global) Gap-Aware master for sm_100a.
//
// Section 5.3 of the paper: G_p = ||theta_p - theta^i_p|| / C_p + 1, one number per layer, and the
// gradient of layer p is multiplied by 1/G_p before the momentum step. The norm is a reduction
// over the layer and must be known before the layer's update, so arrivals cannot be fused in
// time the way the parameter-wise kernel fuses them. Two things can be done instead:
//   * inside one ga_push_batch call the next arriving worker is known, so the pass that applies
//     arrival j also accumulates ||theta_new - theta^{next}||^2 while theta_new is in registers:
//     28 B per parameter per arrival (theta, v, g, next copy in; theta, v, sent copy out) after one
//     distance pass of 8 B per call;
//   * the only thing arrival j+1 needs from arrival j, layer by layer, is that layer's Gap. Each
//     arrival is one launch with one block per tile; a block leaves its tile's partial sums in
//     global memory and takes a ticket of its layer; the block that draws a layer's last ticket sums
//     the layer's partials, does the per-layer step (refresh of m_p, then C_p, G_p, 1/G_p of the next
//     arrival) and advances the layer's epoch counter; a block about to apply the next arrival to
//     a tile first waits for that layer's epoch. Consecutive launches are chained with programmatic
//     dependent launch: every block releases the dependent launch at once, so the next arrival's
//     blocks are scheduled as soon as the current arrival's last blocks have started and fill
//     the SMs that its tail leaves idle -- the epochs, not the launch boundary, carry the ordering,
//     and layers run ahead independently. (A dependent launch only begins once every block of the
//     launch before it is running, so a waiting block can never hold an SM that the block it
//     waits for still needs.)
// A tile is at most kLayerTile consecutive elements of ONE layer (the host cuts the layers into
// tiles), so a block never mixes layers. Squared norms are accumulated in fp64 in a fixed order
// (thread-strided over the tile, warp shuffles, warps in order; tiles of a layer thread-strided in
// index order) and rounded to fp32 once, which makes the result independent of which block happens
// to come last, and reproducible run to run. Data written by one launch and read by the next
// (theta, v, saved copies, the per-layer scalars) is read past the L1 cache, which is not kept
// coherent between SMs. Every wait has an iteration limit, after which the block raises an error
// flag and leaves.
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
    unsigned int* epoch;     // per layer: Gaps made ready so far (distance passes and arrivals), never reset
    int* abort_word;         // set by a block whose wait ran out; ends every later wait at once
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

constexpr unsigned kLayerSpinLimit = 1u << 20;   // polls of a layer's epoch (about a second) before a block gives up

// Waits (thread 0 polls, everybody gets the answer) until the layer's epoch has reached `need`.
// A block whose wait runs out raises the engine's error flag (mapped host memory) and a device-side
// abort word, which every other waiting block sees at its next poll, so one lost dependency ends the
// launches that follow in about a second instead of one time-out per block.
__device__ __forceinline__ bool wait_layer_epoch(const unsigned int* epoch, unsigned int need, int* abort_word, int* err) {
    __shared__ int s_ready;
    if (threadIdx.x == 0) {
        int ready = 0;
        for (unsigned it = 0; it < kLayerSpinLimit; ++it) {
            unsigned int seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(epoch) : "memory");
            if ((int)(seen - need) >= 0) { ready = 1; break; }
            if (*(volatile int*)abort_word) break;
            __nanosleep(64);
        }
        if (!ready) {
            *(volatile int*)abort_word = 1;
            *(volatile int*)err = 2;
            __threadfence_system();
        }
        s_ready = ready;
    }
    __syncthreads();
    return s_ready != 0;
}

// Thread 0 of a layer's last block: the per-layer results are written; let the waiting tiles go.
__device__ __forceinline__ void publish_layer(unsigned int* epoch) {
    __threadfence();
    atomicAdd(epoch, 1u);
}

// ||theta - saved copy||^2 of one tile (the distance pass of a call's first arrival).
__device__ __forceinline__ void dist_tile(const float* __restrict__ theta, const float* __restrict__ saved,
                                          const LayerTables& T, int tile, float inv_bias, const Hyper& h) {
    const Tile t = T.tiles[tile];
    const TileRange r(t);
    double acc = 0.0, none = 0.0;
    auto one = [&](float th, float s) {
        const float diff = __fsub_rn(th, s);
        acc += (double)diff * (double)diff;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) one(__ldcg(theta + i), __ldcg(saved + i));
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        const float4 th = __ldcg(reinterpret_cast<const float4*>(theta + 4 * q));
        const float4 s = __ldcg(reinterpret_cast<const float4*>(saved + 4 * q));
        one(th.x, s.x); one(th.y, s.y); one(th.z, s.z); one(th.w, s.w);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) one(__ldcg(theta + i), __ldcg(saved + i));
    block_sum2(acc, none);
    if (threadIdx.x == 0) T.partial_d[tile] = acc;
    if (!last_tile_of_layer(T, t.layer)) return;
    double tv, td;
    layer_totals(T, t.layer, false, true, tv, td);
    if (threadIdx.x == 0) {
        layer_gap(T, t.layer, td, __ldcg(T.m_layer + t.layer), inv_bias, h);   // m_p may come from another SM
        publish_layer(&T.epoch[t.layer]);
    }
}

// One arrival applied to one tile. next_mode: 0 = the next arrival is not known (last of the call);
// 1 = its worker's saved copy is `next`; 2 = the same worker arrives again, whose copy is the theta
// being saved right now, so its distance is exactly 0. inv_bias_next is 1/(1-beta^k') for the C of
// the next arrival.
__device__ __forceinline__ void update_tile(float* __restrict__ theta, float* __restrict__ vel,
                                            const float* __restrict__ grad, float* __restrict__ saved, int write_saved,
                                            const float* __restrict__ next, int next_mode, const LayerTables& T, int tile,
                                            float eta, const Hyper& h, float inv_bias_next) {
    const Tile t = T.tiles[tile];
    const TileRange r(t);
    const float inv = __ldcg(T.inv_gap + t.layer);     // written by another block during this launch
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
        float th = __ldcg(theta + i), v = __ldcg(vel + i);
        one(th, v, grad[i], look ? __ldcg(next + i) : 0.f);
        theta[i] = th;
        vel[i] = v;
        if (write_saved) saved[i] = th;
    };
    for (long long i = r.b + threadIdx.x; i < r.ab; i += kLayerThreads) scalar(i);
    for (long long q = r.ab / 4 + threadIdx.x; q < r.ae / 4; q += kLayerThreads) {
        float4 th = __ldcg(reinterpret_cast<const float4*>(theta + 4 * q));
        float4 v = __ldcg(reinterpret_cast<const float4*>(vel + 4 * q));
        const float4 g = ld_stream(grad + 4 * q);
        const float4 s = look ? __ldcg(reinterpret_cast<const float4*>(next + 4 * q)) : make_float4(0.f, 0.f, 0.f, 0.f);
        one(th.x, v.x, g.x, s.x); one(th.y, v.y, g.y, s.y); one(th.z, v.z, g.z, s.z); one(th.w, v.w, g.w, s.w);
        *reinterpret_cast<float4*>(theta + 4 * q) = th;
        *reinterpret_cast<float4*>(vel + 4 * q) = v;
        if (write_saved) st_stream(saved + 4 * q, th);
    }
    for (long long i = r.ae + threadIdx.x; i < r.e; i += kLayerThreads) scalar(i);
    block_sum2(acc_v, acc_d);
    if (threadIdx.x == 0) {
        T.partial_v[tile] = acc_v;
        T.partial_d[tile] = acc_d;
    }
    if (!last_tile_of_layer(T, t.layer)) return;
    double tv, td;
    layer_totals(T, t.layer, true, look, tv, td);
    if (threadIdx.x == 0) {
        const float m_new = __fmaf_rn(h.beta, __ldcg(T.m_layer + t.layer), __fmul_rn(h.one_minus_beta, (float)tv));
        T.m_layer[t.layer] = m_new;
        if (next_mode != 0) layer_gap(T, t.layer, td, m_new, inv_bias_next, h);   // mode 2: td = 0
        publish_layer(&T.epoch[t.layer]);
    }
}

// Lets the launch that depends on this one begin as soon as all blocks of this one are running.
__device__ __forceinline__ void release_dependent_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// First arrival of a call: the distance pass, one block per tile; ends with every layer's Gap.
__global__ void __launch_bounds__(kLayerThreads)
ga_layer_dist_kernel(const float* __restrict__ theta, const float* __restrict__ saved, LayerTables T, float inv_bias,
                     const __grid_constant__ Hyper h) {
    release_dependent_launch();
    dist_tile(theta, saved, T, blockIdx.x, inv_bias, h);
}

// One arrival, one block per tile. `need` is the epoch value at which this arrival's Gap of a layer
// is in place. The launch before it may still be running: the wait on the tile's layer orders this
// block after everything it reads.
__global__ void __launch_bounds__(kLayerThreads)
ga_layer_arrival_kernel(float* __restrict__ theta, float* __restrict__ vel, const float* __restrict__ grad,
                        float* __restrict__ saved, int write_saved, const float* __restrict__ next, int next_mode,
                        unsigned int need, LayerTables T, float eta, const __grid_constant__ Hyper h, float inv_bias_next,
                        int* err) {
    release_dependent_launch();
    if (!wait_layer_epoch(&T.epoch[T.tiles[blockIdx.x].layer], need, T.abort_word, err)) return;
    update_tile(theta, vel, grad, saved, write_saved, next, next_mode, T, blockIdx.x, eta, h, inv_bias_next);
}

// One block that waits for an epoch nobody advances: the wait must run out, raise the flag and let the
// block return (ga_selftest_bounded_wait).
__global__ void __launch_bounds__(kLayerThreads)
ga_layer_wait_probe_kernel(const unsigned int* epoch, int* abort_word, int* err, int* gave_up) {
    const bool ready = wait_layer_epoch(epoch, 1u, abort_word, err);
    if (threadIdx.x == 0) *gave_up = ready ? 0 : 1;
}

}  // namespace ga
