// Host side of the C ABI declared in include/ga.h: argument checks, the master's integer
// bookkeeping (arrival counter, iter[], delays, bias-correction scalars, window cutting) and
// kernel launches. All arithmetic on parameters happens in the kernels of ga_kernels.cuh.
#include "ga.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "ga_kernels.cuh"
#include "ga_layer_kernels.cuh"
#include "ga_selftest.cuh"

namespace {

thread_local std::string g_error;

int fail(int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_error = buf;
    return code;
}

constexpr long long kRowAlign = 32;            // floats: rows start on 128-byte boundaries
#ifndef GA_HOST_CHUNK_FLOATS
#define GA_HOST_CHUNK_FLOATS (4ll << 20)
#endif
#ifndef GA_HOST_STAGES
#define GA_HOST_STAGES 2
#endif
constexpr long long kHostChunk = GA_HOST_CHUNK_FLOATS;   // floats per chunk of the host-buffer path
constexpr int kHostStages = GA_HOST_STAGES;              // staging buffers the copies-in rotate through
constexpr int kHostD2hRing = 4;                // chunks the kernels may run ahead of the copies out
constexpr int kLayerHostGroup = 1;             // whole gradient vectors per staging buffer (layer-wise Gap)
constexpr uint32_t kStateMagic = 0x47415331;   // "GAS1"
constexpr int kStatsLog = GA_STATS_LOG;        // arrivals whose Gap statistics are kept

}  // namespace

struct ga_engine {
    long long d = 0, stride = 0;  // parameters; padded row length in floats
    int n_workers = 0, variant = GA_GA, device = 0;
    float lr = 0, lr_max = 0, gamma = 0, beta = 0, eps = 1e-8f;   // lr = eta_k, lr_max = eta_max of C
    int c_order = 0, fast_math = 0, stats = 0, window = GA_MAX_WINDOW;
    float *theta = nullptr, *vel = nullptr, *mom = nullptr, *saved = nullptr;
    float* vworker = nullptr;     // DANA: N rows, v^i of every worker (vel then holds their sum)
    // layer-wise Gap: layers cut into tiles, one scalar m_p / Gap / 1/Gap per layer
    std::vector<int64_t> layer_off;
    ga::Tile* tiles = nullptr;
    int* tile_begin = nullptr;     // n_layers + 1
    double* tile_partial = nullptr;   // 2 x n_tiles: sums of v^2, then sums of squared distances
    unsigned int* layer_ticket = nullptr;
    unsigned int* layer_epoch = nullptr;   // per layer: Gaps made ready so far; layer_epoch_host mirrors their common value
    int* layer_abort = nullptr;            // device word: a wait of the layer kernels ran out
    unsigned int layer_epoch_host = 0;
    float *m_layer = nullptr, *layer_gap = nullptr, *layer_inv_gap = nullptr;
    int n_tiles = 0;
    ga::LayerTables layer_tables() const {
        return ga::LayerTables{tiles, tile_begin, tile_partial, tile_partial + n_tiles, layer_ticket, layer_epoch,
                               layer_abort, m_layer, layer_gap, layer_inv_gap};
    }
    bool is_layer() const { return variant == GA_GA_LAYER; }
    int n_layers() const { return (int)layer_off.size() - 1; }
    float* sec = nullptr;         // Adam: second moment (vel holds the first moment, gamma is beta_1)
    float beta2 = 0.999f, adam_eps = 1e-8f;
    float weight_decay = 0.f;
    int nesterov = 0;
    std::vector<int64_t> iter;
    int64_t k_done = 0, k_c = 0;
    cudaStream_t stream = nullptr;
    bool cuda_failed = false;
    bool owns_state = true;        // false: theta, v, m, the copies and the statistics buffers live in the caller's workspace
    // statistics
    ga::StatsPartial* partials = nullptr;
    double* stats_dev = nullptr;   // ring of kStatsLog x {sum, max}: one pair per arrival
    int stats_blocks = 0;
    int sms = 148;                 // multiprocessors of the engine's device
    int small_range_vectors = 0;   // ranges of fewer 16-byte vectors than this run with two parameters per thread
    int64_t stats_total = 0;       // arrivals logged since the current call began (slot = index % kStatsLog)
    const void* known_dev_ptrs[64] = {};   // caller's device pointers already looked up (check_dev_ptr)
    unsigned known_dev_next = 0;
    // pull kernel error flag: one int of pinned, device-mapped host memory
    int* pull_err = nullptr;
    // beta^k, gamma^k, beta2^k carried from one arrival to the next (see inv_one_minus_pow)
    struct PowCache { double base = 0.0, p = 0.0; int64_t k = -1; };
    PowCache pow_c, pow_b1, pow_b2;
    // host-buffer path
    float* stage[kHostStages] = {};
    long long stage_elems = 0;
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
    cudaEvent_t ev_h2d[kHostStages] = {}, ev_kernel[kHostStages] = {}, ev_prev = nullptr;
    cudaEvent_t ev_d2h[kHostD2hRing] = {};

    float* row(int i) const { return saved + (size_t)i * stride; }
    float* vrow(int i) const { return vworker ? vworker + (size_t)i * stride : nullptr; }
    bool is_dana() const { return variant == GA_DANA || variant == GA_DANA_SA || variant == GA_DANA_GA; }
    bool is_adam() const { return variant == GA_ADAM || variant == GA_ADAM_SA || variant == GA_ADAM_GA; }
    bool is_gap() const { return variant == GA_GA || variant == GA_GA_LAYER || variant == GA_DANA_GA || variant == GA_ADAM_GA; }
    bool is_tau_grad() const { return variant == GA_SA_GRAD || variant == GA_DANA_SA || variant == GA_ADAM_SA; }
    ga::Hyper hyper() const {
        ga::Hyper h;
        h.eta_max = lr_max;
        h.gamma = gamma;
        h.beta = beta;
        h.one_minus_beta = (float)(1.0 - (double)beta);
        h.eps = eps;
        h.eta_gamma = lr * gamma;
        h.one_minus_gamma = (float)(1.0 - (double)gamma);
        h.beta2 = beta2;
        h.one_minus_beta2 = (float)(1.0 - (double)beta2);
        h.adam_eps = adam_eps;
        h.wd = weight_decay;
        h.nesterov = nesterov;
        h.short_forms = ga::short_forms_ok(lr_max, eps, is_adam() ? adam_eps : 1e-8f,
                                           is_adam() ? h.one_minus_gamma : 1.0f) ? 1 : 0;
        return h;
    }
    // (float)(1 / (1 - base^k)), base^k = pow(base, k) in double. Consecutive k reuse the previous
    // power: p = p_prev * base drifts from pow() by far less than 1e-13 relative between the
    // re-synchronisations every 64 steps, and the result is monotone in p, so whenever both
    // ends of p (1 -+ 1e-13) round to the same float that float is also what pow() gives;
    // otherwise pow() itself decides.
    static float inv_one_minus_pow(PowCache& c, double base, int64_t k) {
        if (c.k >= 0 && c.base == base && k == c.k + 1 && (k & 63) != 0) {
            const double p = c.p * base;
            c.p = p;
            c.k = k;
            const float lo = (float)(1.0 / (1.0 - p * (1.0 - 1e-13)));
            const float hi = (float)(1.0 / (1.0 - p * (1.0 + 1e-13)));
            if (lo == hi) return lo;
        }
        c.base = base;
        c.k = k;
        c.p = std::pow(base, (double)k);
        return (float)(1.0 / (1.0 - c.p));
    }
    // 1/(1-beta^k) for the C in force after k refreshes of m; 0 before the first (C = eta_max*eps)
    float inv_bias(int64_t k) {
        if (k <= 0) return 0.f;
        return inv_one_minus_pow(pow_c, (double)beta, k);
    }
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

int cuda_fail(ga_engine* e, cudaError_t err, const char* what) {
    if (e) e->cuda_failed = true;
    return fail(GA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(err));
}

#define GA_CUDA(e, call)                                             \
    do {                                                             \
        cudaError_t err__ = (call);                                  \
        if (err__ != cudaSuccess) return cuda_fail((e), err__, #call); \
    } while (0)

int check_engine(ga_engine* e) {
    if (!e) return fail(GA_ERR_ARG, "engine is NULL");
    if (e->cuda_failed) return fail(GA_ERR_CUDA, "engine is unusable after an earlier CUDA error");
    return GA_OK;
}

int check_worker(ga_engine* e, int worker) {
    if (worker < 0 || worker >= e->n_workers)
        return fail(GA_ERR_ARG, "worker %d out of range [0, %d)", worker, e->n_workers);
    return GA_OK;
}

int check_dev_ptr(const void* p, const char* name) {
    if (!p) return fail(GA_ERR_ARG, "%s is NULL", name);
    if ((uintptr_t)p % 16) return fail(GA_ERR_ARG, "%s is not 16-byte aligned", name);
    return GA_OK;
}

// The same for an engine's call, plus: is this memory a kernel of the engine's device can read? A
// pointer to ordinary host memory handed over as a device pointer would fault the kernel that
// dereferences it, so the runtime is asked once per pointer (callers reuse their gradient buffers:
// the last 64 accepted pointers are remembered). Pinned or managed memory passes: the device can reach it.
bool known_dev_ptr(const ga_engine* e, const void* p) {
    for (const void* seen : e->known_dev_ptrs)
        if (seen == p) return true;
    return false;
}

int check_dev_ptr(ga_engine* e, const void* p, const char* name) {
    if (int rc = check_dev_ptr(p, name)) return rc;
    if (known_dev_ptr(e, p)) return GA_OK;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        cudaGetLastError();
        return fail(GA_ERR_ARG, "%s is not memory the CUDA runtime knows", name);
    }
    if (attr.type == cudaMemoryTypeUnregistered)
        return fail(GA_ERR_ARG, "%s points to ordinary host memory, not to device memory", name);
    if (attr.type == cudaMemoryTypeDevice && attr.device != e->device) {
        int reachable = 0;
        cudaDeviceCanAccessPeer(&reachable, e->device, attr.device);
        if (!reachable) return fail(GA_ERR_ARG, "%s lives on device %d, which device %d cannot reach", name, attr.device, e->device);
    }
    e->known_dev_ptrs[e->known_dev_next++ % (sizeof e->known_dev_ptrs / sizeof e->known_dev_ptrs[0])] = p;
    return GA_OK;
}

// Every synchronising call ends here: wait for the engine's stream, then see whether a bounded
// wait inside a kernel ran out (a bulk copy of the pull kernel, or a layer's Gap in the layer-wise
// kernel): the kernel then raised a flag in mapped host memory and left its work incomplete, so
// the failure is sticky like a CUDA error.
int sync_and_check(ga_engine* e) {
    GA_CUDA(e, cudaStreamSynchronize(e->stream));
    if (const int flag = *(volatile int*)e->pull_err) {
        e->cuda_failed = true;
        return fail(GA_ERR_CUDA, flag == 2 ? "a block of the layer-wise kernel gave up waiting for a layer's Gap"
                                           : "a bulk copy of ga_pull did not complete within its wait limit");
    }
    return GA_OK;
}

int grid_1d(long long n, int threads, int cap) {
    long long g = (n + threads - 1) / threads;
    if (g < 1) g = 1;
    return (int)(g < cap ? g : cap);
}

// ----------------------------------------------------------------------------- launch

// A launch that may be scheduled while the one before it on the stream is still draining (programmatic
// dependent launch). The window kernel then waits for that launch to complete before it touches
// memory; the layer kernels order themselves through the layers' epoch counters instead.
template <typename... Params, typename... Args>
cudaError_t launch_chained(void (*kernel)(Params...), long long grid, int block, cudaStream_t st, bool chained, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

// stats_mode (STATS instantiations): 1 = the arrivals' pairs overwrite their log slots, 2 = they are
// merged into them (a later chunk of the same arrivals on the host-buffer path)
template <int FAMILY, int PENALTY, bool EXACT, int C_ORDER, bool STATS>
void launch_window_t(ga_engine* e, const ga::Window& w, long long vec_begin, long long vec_end, cudaStream_t st,
                     int stats_mode) {
    // vec_begin / vec_end count 16-byte vectors (four parameters). A range too short to give every SM
    // a full set of blocks at four parameters per thread runs with two per thread instead: twice the
    // warps to hide an arrival's dependent chain behind, which is what bounds an L2-resident vector.
    const bool narrow = (vec_end - vec_begin) < (long long)e->small_range_vectors;
    const long long first = narrow ? vec_begin * 2 : vec_begin, last = narrow ? vec_end * 2 : vec_end;
    long long blocks = (last - first + ga::kThreads - 1) / ga::kThreads;
    if (STATS && blocks > e->stats_blocks) blocks = e->stats_blocks;
    // a single arrival has nothing to prefetch across: the one-arrival instantiation is leaner.
    constexpr int ST = GA_WINDOW_STAGES;
    // launched so that it may be scheduled under the tail of the launch before it (the kernel waits for
    // that launch to complete before its first access to global memory)
#define GA_LAUNCH_V(BATCH, STAGES_, WD_, VEC_)                                                                       \
    launch_chained(ga::ga_window_kernel<FAMILY, PENALTY, EXACT, C_ORDER, STATS, BATCH, STAGES_, WD_, VEC_>,           \
                   (long long)blocks, ga::kThreads, st, true, e->theta, e->vel, e->mom, e->sec, w, e->hyper(), first, \
                   last, e->d, e->partials)
#define GA_LAUNCH(BATCH, STAGES_, WD_) \
    do { if (narrow) GA_LAUNCH_V(BATCH, STAGES_, WD_, 2); else GA_LAUNCH_V(BATCH, STAGES_, WD_, 4); } while (0)
    const bool wd = e->weight_decay != 0.f || e->nesterov;   // the instantiations with the extras
    if (w.K == 1) { if (wd) GA_LAUNCH(1, 0, true); else GA_LAUNCH(1, 0, false); }
    else { if (wd) GA_LAUNCH(GA_WINDOW_BATCH, ST, true); else GA_LAUNCH(GA_WINDOW_BATCH, ST, false); }
#undef GA_LAUNCH
#undef GA_LAUNCH_V
    if (STATS) {
        ga::ga_stats_finish_kernel<<<w.K, 256, 0, st>>>(e->partials, (int)blocks, e->stats_dev, e->stats_total,
                                                        kStatsLog, stats_mode == 2);
    }
}

template <int FAMILY>
void launch_family(ga_engine* e, const ga::Window& w, long long vb, long long ve, cudaStream_t st, int stats) {
    if (e->is_gap()) {
        const bool exact = !e->fast_math;
#define GA_CASE(EX, CO, ST) launch_window_t<FAMILY, ga::PEN_GAP, EX, CO, ST>(e, w, vb, ve, st, stats)
        if (exact) {
            if (e->c_order == 0) { if (stats) GA_CASE(true, 0, true); else GA_CASE(true, 0, false); }
            else { if (stats) GA_CASE(true, 1, true); else GA_CASE(true, 1, false); }
        } else {
            if (e->c_order == 0) { if (stats) GA_CASE(false, 0, true); else GA_CASE(false, 0, false); }
            else { if (stats) GA_CASE(false, 1, true); else GA_CASE(false, 1, false); }
        }
#undef GA_CASE
    } else if (e->is_tau_grad()) {
        launch_window_t<FAMILY, ga::PEN_TAU, true, 0, false>(e, w, vb, ve, st, 0);
    } else {
        launch_window_t<FAMILY, ga::PEN_NONE, true, 0, false>(e, w, vb, ve, st, 0);
    }
}

// One launch for arrivals w over vectors [vec_begin, vec_end). first_range / last_range say whether
// this range is the first / last of the arrivals' parameter ranges (both true for a whole vector):
// the Gap statistics of an arrival are complete, and counted, once its last range has run.
int launch_window(ga_engine* e, const ga::Window& w, long long vec_begin, long long vec_end, cudaStream_t st,
                  bool first_range = true, bool last_range = true) {
    if (vec_end <= vec_begin || w.K <= 0) return GA_OK;
    if (e->is_layer()) return fail(GA_ERR_STATE, "the layer-wise Gap takes whole arrivals: see launch_layer_arrivals");
    const int stats = (e->stats && e->is_gap()) ? (first_range ? 1 : 2) : 0;
    if (e->is_dana()) launch_family<ga::DANA>(e, w, vec_begin, vec_end, st, stats);
    else if (e->is_adam()) launch_family<ga::ADAM>(e, w, vec_begin, vec_end, st, stats);
    else launch_family<ga::MOM>(e, w, vec_begin, vec_end, st, stats);
    GA_CUDA(e, cudaGetLastError());
    if (stats && last_range) e->stats_total += w.K;
    return GA_OK;
}

void free_layers(ga_engine* e) {
    cudaFree(e->tiles); cudaFree(e->tile_begin); cudaFree(e->tile_partial); cudaFree(e->layer_ticket);
    cudaFree(e->layer_epoch);
    cudaFree(e->layer_abort);
    e->layer_epoch = nullptr;
    e->layer_abort = nullptr;
    cudaFree(e->m_layer); cudaFree(e->layer_gap); cudaFree(e->layer_inv_gap);
    e->tiles = nullptr; e->tile_begin = nullptr; e->tile_partial = nullptr; e->layer_ticket = nullptr;
    e->m_layer = e->layer_gap = e->layer_inv_gap = nullptr;
    e->n_tiles = 0;
}

// Cut the layers into tiles and put the tables on the device. offsets: n + 1 entries.
int build_layers(ga_engine* e, const int64_t* offsets, int n) {
    std::vector<ga::Tile> tiles;
    std::vector<int> begin(n + 1);
    for (int p = 0; p < n; ++p) {
        begin[p] = (int)tiles.size();
        for (int64_t at = offsets[p]; at < offsets[p + 1]; at += ga::kLayerTile) {
            ga::Tile t;
            t.start = at;
            t.len = (int)std::min<int64_t>(ga::kLayerTile, offsets[p + 1] - at);
            t.layer = p;
            tiles.push_back(t);
        }
    }
    begin[n] = (int)tiles.size();
    free_layers(e);
    const size_t nt = tiles.size();
    bool ok = cudaMalloc(&e->tiles, sizeof(ga::Tile) * nt) == cudaSuccess &&
              cudaMalloc(&e->tile_begin, sizeof(int) * (n + 1)) == cudaSuccess &&
              cudaMalloc(&e->tile_partial, sizeof(double) * 2 * nt) == cudaSuccess &&
              cudaMalloc(&e->layer_ticket, sizeof(unsigned int) * n) == cudaSuccess &&
              cudaMalloc(&e->layer_epoch, sizeof(unsigned int) * n) == cudaSuccess &&
              cudaMalloc(&e->layer_abort, sizeof(int)) == cudaSuccess &&
              cudaMalloc(&e->m_layer, sizeof(float) * n) == cudaSuccess &&
              cudaMalloc(&e->layer_gap, sizeof(float) * n) == cudaSuccess &&
              cudaMalloc(&e->layer_inv_gap, sizeof(float) * n) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_layers(e);
        return fail(GA_ERR_OOM, "cannot allocate the layer tables");
    }
    GA_CUDA(e, cudaMemcpy(e->tiles, tiles.data(), sizeof(ga::Tile) * nt, cudaMemcpyHostToDevice));
    GA_CUDA(e, cudaMemcpy(e->tile_begin, begin.data(), sizeof(int) * (n + 1), cudaMemcpyHostToDevice));
    GA_CUDA(e, cudaMemset(e->m_layer, 0, sizeof(float) * n));
    GA_CUDA(e, cudaMemset(e->layer_gap, 0, sizeof(float) * n));
    GA_CUDA(e, cudaMemset(e->layer_ticket, 0, sizeof(unsigned int) * n));
    GA_CUDA(e, cudaMemset(e->layer_epoch, 0, sizeof(unsigned int) * n));
    GA_CUDA(e, cudaMemset(e->layer_abort, 0, sizeof(int)));
    e->layer_epoch_host = 0;

    e->layer_off.assign(offsets, offsets + n + 1);
    e->n_tiles = (int)nt;
    return GA_OK;
}

// Arrivals w.K of a window with the layer-wise Gap, one launch each, chained. The Gap of the
// window's first arrival is in place already when `primed` (the launch before prepared it);
// otherwise a distance pass computes it first. `next_row` / `next_inv_bias` describe the arrival
// that follows the window inside the same call (nullptr: none is known), so that the window's last
// arrival can prepare its Gap as well.
int launch_layer_arrivals(ga_engine* e, const ga::Window& w, bool primed, const float* next_row, float next_inv_bias) {
    const ga::Hyper h = e->hyper();
    const ga::LayerTables T = e->layer_tables();
    if (!primed) {   // opens a call: ordinary launch, after everything already on the stream
        GA_CUDA(e, launch_chained(ga::ga_layer_dist_kernel, e->n_tiles, ga::kLayerThreads, e->stream, false, e->theta,
                                  w.saved[0], T, w.inv_bias[0], h));
        e->layer_epoch_host += 1;
    }
    for (int j = 0; j < w.K; ++j) {
        const float* nxt = j + 1 < w.K ? w.saved[j + 1] : next_row;
        const float nxt_ib = j + 1 < w.K ? w.inv_bias[j + 1] : next_inv_bias;
        // the same worker again right away: its saved copy is the theta this launch writes, distance 0
        const int mode = !nxt ? 0 : (nxt == w.saved[j] && w.write_saved) ? 2 : 1;
        GA_CUDA(e, launch_chained(ga::ga_layer_arrival_kernel, e->n_tiles, ga::kLayerThreads, e->stream, true, e->theta,
                                  e->vel, w.grad[j], w.saved[j], w.write_saved, nxt, mode, e->layer_epoch_host, T, e->lr, h,
                                  nxt_ib, e->pull_err));
        e->layer_epoch_host += 1;   // every arrival advances every layer's epoch once
    }
    return GA_OK;
}

// Fill the arrival table for arrivals j0..j0+K-1 of a batch and advance the counters.
void fill_window(ga_engine* e, ga::Window& w, const int* workers, const float* const* grads, int K,
                 bool with_pull, int64_t* delays) {
    w.K = K;
    w.write_saved = with_pull ? 1 : 0;
    w.grad_offset = 0;
    for (int j = 0; j < K; ++j) {
        const int i = workers[j];
        const int64_t k = e->k_done + 1;
        const int64_t tau = k - e->iter[i];
        if (delays) delays[j] = tau;
        w.grad[j] = grads[j];
        w.saved[j] = e->row(i);
        w.vworker[j] = e->vrow(i);
        w.tau[j] = (float)tau;
        w.inv_tau[j] = 1.0f / (float)tau;   // IEEE division on the host = the correctly rounded reciprocal
        w.bias1[j] = w.bias2[j] = 1.f;
        if (e->is_adam()) {   // Adam's bias corrections use the arrival index
            w.bias1[j] = ga_engine::inv_one_minus_pow(e->pow_b1, (double)e->gamma, k);
            w.bias2[j] = ga_engine::inv_one_minus_pow(e->pow_b2, (double)e->beta2, k);
        }
        w.eta_eff[j] = e->variant == GA_SA ? e->lr / (float)tau : e->lr;
        if (e->is_gap()) {
            // the C in force for this arrival: after k_c refreshes (lagged order), or after
            // this arrival's own refresh (Adam order)
            w.inv_bias[j] = e->inv_bias(e->c_order == 0 ? e->k_c : e->k_c + 1);
            e->k_c += 1;
        } else {
            w.inv_bias[j] = 0.f;
        }
        e->k_done = k;
        if (with_pull) e->iter[i] = k;
    }
    for (int j = K; j < ga::kMaxWindow; ++j) {
        w.grad[j] = nullptr;
        w.saved[j] = nullptr;
        w.vworker[j] = nullptr;
        w.tau[j] = 1.f;
        w.inv_tau[j] = 1.f;
        w.bias1[j] = w.bias2[j] = 1.f;
        w.inv_bias[j] = 0.f;
        w.eta_eff[j] = 0.f;
    }
}

// Length of the next window starting at schedule[pos]: at most `window` arrivals, cut where a
// worker would appear a second time.
int next_window(const int* schedule, int pos, int K, int window) {
    int n = 0;
    while (pos + n < K && n < window) {
        bool repeat = false;
        for (int q = 0; q < n; ++q) repeat |= schedule[pos + q] == schedule[pos + n];
        if (repeat) break;
        ++n;
    }
    return n;
}

int validate_batch(ga_engine* e, const int* schedule, const void* const* bufs, int K, bool device_ptrs) {
    if (K < 0) return fail(GA_ERR_ARG, "K = %d is negative", K);
    if (K > 0 && (!schedule || !bufs)) return fail(GA_ERR_ARG, "schedule or gradient array is NULL");
    for (int j = 0; j < K; ++j) {
        if (int rc = check_worker(e, schedule[j])) return rc;
        if (!bufs[j]) return fail(GA_ERR_ARG, "gradient %d is NULL", j);
        if (device_ptrs && ((uintptr_t)bufs[j] % 16 || !known_dev_ptr(e, bufs[j]))) {   // not seen before: the full check
            char name[32];
            snprintf(name, sizeof name, "gradient %d", j);
            if (int rc = check_dev_ptr(e, bufs[j], name)) return rc;
        }
    }
    return GA_OK;
}

int ensure_host_path(ga_engine* e) {
    if (e->stage[0]) return GA_OK;
    // parameter-wise masters stage a chunk of every gradient of a window; the layer-wise Gap needs
    // whole vectors before a layer's norm is known, so it stages a few whole gradients instead
    const long long chunk = e->is_layer() ? e->stride : (e->stride < kHostChunk ? e->stride : kHostChunk);
    const int per_stage = e->is_layer() ? kLayerHostGroup : ga::kMaxWindow;
    e->stage_elems = chunk;
    for (int s = 0; s < kHostStages; ++s) {
        if (cudaMalloc(&e->stage[s], sizeof(float) * (size_t)chunk * per_stage) != cudaSuccess) {
            cudaGetLastError();
            return fail(GA_ERR_OOM, "cannot allocate staging buffers for the host-buffer path");
        }
        GA_CUDA(e, cudaEventCreateWithFlags(&e->ev_h2d[s], cudaEventDisableTiming));
        GA_CUDA(e, cudaEventCreateWithFlags(&e->ev_kernel[s], cudaEventDisableTiming));
    }
    GA_CUDA(e, cudaEventCreateWithFlags(&e->ev_prev, cudaEventDisableTiming));
    for (int q = 0; q < kHostD2hRing; ++q) GA_CUDA(e, cudaEventCreateWithFlags(&e->ev_d2h[q], cudaEventDisableTiming));
    GA_CUDA(e, cudaStreamCreateWithFlags(&e->s_h2d, cudaStreamNonBlocking));
    GA_CUDA(e, cudaStreamCreateWithFlags(&e->s_d2h, cudaStreamNonBlocking));
    return GA_OK;
}

}  // namespace

// ================================================================================= C ABI
extern "C" {

const char* ga_last_error(void) { return g_error.c_str(); }

}  // extern "C"

namespace {

constexpr int kMaxStatsBlocks = 2048;   // the workspace reserves room for this many per-block partials per arrival

bool is_dana_variant(int v) { return v == GA_DANA || v == GA_DANA_SA || v == GA_DANA_GA; }
bool is_adam_variant(int v) { return v == GA_ADAM || v == GA_ADAM_SA || v == GA_ADAM_GA; }

// Where everything of fixed size lives inside one device allocation (offsets in bytes, 256-byte aligned).
struct StatePlan {
    size_t theta, vel, mom, saved, vworker, sec, partials, stats, total;
};

StatePlan plan_state(long long stride, int n_workers, int variant) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t row = up(sizeof(float) * (size_t)stride);   // rows are multiples of 128 bytes already
    StatePlan p{};
    size_t at = 0;
    p.theta = at; at += row;
    p.vel = at; at += row;
    p.mom = at; at += row;
    p.saved = at; at += up(sizeof(float) * (size_t)stride * (size_t)n_workers);
    p.vworker = at; if (is_dana_variant(variant)) at += up(sizeof(float) * (size_t)stride * (size_t)n_workers);
    p.sec = at; if (is_adam_variant(variant)) at += row;
    p.partials = at; at += up(sizeof(ga::StatsPartial) * (size_t)kMaxStatsBlocks * ga::kMaxWindow);
    p.stats = at; at += up(sizeof(double) * 2 * kStatsLog);
    p.total = at;
    return p;
}

long long padded_stride(size_t n_params) { return ((long long)n_params + kRowAlign - 1) / kRowAlign * kRowAlign; }

// ga_create and ga_create_in: workspace == nullptr lets the engine allocate its own state.
ga_engine* create_engine(size_t n_params, int n_workers, float lr, float momentum, float c_beta, int variant,
                         void* workspace, size_t workspace_bytes, bool in_workspace) {
    g_error.clear();
    if (n_params == 0 || n_params > (size_t)1 << 34) { fail(GA_ERR_ARG, "n_params out of range"); return nullptr; }
    if (n_workers <= 0 || n_workers > 65536) { fail(GA_ERR_ARG, "n_workers out of range"); return nullptr; }
    if (!(lr > 0.f) || !std::isfinite(lr)) { fail(GA_ERR_ARG, "lr must be positive and finite"); return nullptr; }
    if (!(lr * 1e-8f > 0.f)) {   // C = eta_max (sqrt(m_hat) + eps) must stay positive: a Gap of x/0 has no meaning
        fail(GA_ERR_ARG, "lr is so small that lr * 1e-8 (the smallest C) rounds to zero");
        return nullptr;
    }
    if (!(std::fabs(momentum) < 1.f)) { fail(GA_ERR_ARG, "|momentum| must be < 1"); return nullptr; }
    if (!(c_beta >= 0.f && c_beta < 1.f)) { fail(GA_ERR_ARG, "c_beta must be in [0, 1)"); return nullptr; }
    if (variant < GA_ASGD || variant > GA_GA_LAYER) { fail(GA_ERR_ARG, "unknown variant %d", variant); return nullptr; }
    ga_engine* e = new (std::nothrow) ga_engine();
    if (!e) { fail(GA_ERR_OOM, "out of host memory"); return nullptr; }
    e->d = (long long)n_params;
    e->stride = (e->d + kRowAlign - 1) / kRowAlign * kRowAlign;
    e->n_workers = n_workers;
    e->lr = lr;
    e->lr_max = lr;
    e->gamma = momentum;
    e->beta = c_beta;
    e->variant = variant;
    e->iter.assign(n_workers, 0);
    if (cudaGetDevice(&e->device) != cudaSuccess) {
        fail(GA_ERR_CUDA, "no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
        delete e;
        return nullptr;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, e->device) == cudaSuccess) e->sms = prop.multiProcessorCount;
    const int sms = e->sms;
    e->stats_blocks = sms * 8 < kMaxStatsBlocks ? sms * 8 : kMaxStatsBlocks;
    e->small_range_vectors = sms * 9 * ga::kThreads;   // one full set of resident blocks at four parameters per thread
    const size_t row_bytes = sizeof(float) * (size_t)e->stride;
    bool ok;
    if (in_workspace) {   // carve the caller's memory; nothing of it is ever freed here
        const StatePlan p = plan_state(e->stride, n_workers, variant);
        if (!workspace || (uintptr_t)workspace % 256 || workspace_bytes < p.total) {
            fail(GA_ERR_ARG, "workspace must be 256-byte aligned device memory of at least %zu bytes (ga_workspace_bytes)", p.total);
            delete e;
            return nullptr;
        }
        char* base = (char*)workspace;
        e->owns_state = false;
        e->theta = (float*)(base + p.theta);
        e->vel = (float*)(base + p.vel);
        e->mom = (float*)(base + p.mom);
        e->saved = (float*)(base + p.saved);
        if (e->is_dana()) e->vworker = (float*)(base + p.vworker);
        if (e->is_adam()) e->sec = (float*)(base + p.sec);
        e->partials = (ga::StatsPartial*)(base + p.partials);
        e->stats_dev = (double*)(base + p.stats);
        ok = cudaHostAlloc(&e->pull_err, sizeof(int), cudaHostAllocMapped) == cudaSuccess;
    } else {
        ok = cudaMalloc(&e->theta, row_bytes) == cudaSuccess && cudaMalloc(&e->vel, row_bytes) == cudaSuccess &&
             cudaMalloc(&e->mom, row_bytes) == cudaSuccess &&
             cudaMalloc(&e->saved, row_bytes * (size_t)n_workers) == cudaSuccess &&
             cudaMalloc(&e->partials, sizeof(ga::StatsPartial) * (size_t)e->stats_blocks * ga::kMaxWindow) == cudaSuccess &&
             cudaMalloc(&e->stats_dev, sizeof(double) * 2 * kStatsLog) == cudaSuccess &&
             cudaHostAlloc(&e->pull_err, sizeof(int), cudaHostAllocMapped) == cudaSuccess &&
             (!e->is_dana() || cudaMalloc(&e->vworker, row_bytes * (size_t)n_workers) == cudaSuccess) &&
             (!e->is_adam() || cudaMalloc(&e->sec, row_bytes) == cudaSuccess);
    }
    if (ok) {
        ok = cudaMemset(e->theta, 0, row_bytes) == cudaSuccess && cudaMemset(e->vel, 0, row_bytes) == cudaSuccess &&
             cudaMemset(e->mom, 0, row_bytes) == cudaSuccess &&
             cudaMemset(e->saved, 0, row_bytes * (size_t)n_workers) == cudaSuccess &&
             (*e->pull_err = 0, true) &&
             (!e->vworker || cudaMemset(e->vworker, 0, row_bytes * (size_t)n_workers) == cudaSuccess) &&
             (!e->sec || cudaMemset(e->sec, 0, row_bytes) == cudaSuccess) &&
             cudaFuncSetAttribute(ga::ga_pull_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  ga::kPullStages * ga::kPullChunk) == cudaSuccess &&
             cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        cudaError_t err = cudaGetLastError();
        fail(err == cudaErrorMemoryAllocation ? GA_ERR_OOM : GA_ERR_CUDA, "ga_create: %s", cudaGetErrorString(err));
        ga_destroy(e);
        return nullptr;
    }
    if (e->is_layer()) {   // until ga_set_layers says otherwise: one layer, the global Gap
        const int64_t whole[2] = {0, e->d};
        if (build_layers(e, whole, 1) != GA_OK) { ga_destroy(e); return nullptr; }
    }
    return e;
}

}  // namespace

extern "C" {

ga_engine* ga_create(size_t n_params, int n_workers, float lr, float momentum, float c_beta, int variant) {
    return create_engine(n_params, n_workers, lr, momentum, c_beta, variant, nullptr, 0, false);
}

size_t ga_workspace_bytes(size_t n_params, int n_workers, int variant) {
    if (n_params == 0 || n_params > (size_t)1 << 34 || n_workers <= 0 || n_workers > 65536 || variant < GA_ASGD ||
        variant > GA_GA_LAYER) {
        fail(GA_ERR_ARG, "ga_workspace_bytes: arguments out of range");
        return 0;
    }
    return plan_state(padded_stride(n_params), n_workers, variant).total;
}

ga_engine* ga_create_in(size_t n_params, int n_workers, float lr, float momentum, float c_beta, int variant,
                        void* workspace_dev, size_t workspace_bytes) {
    return create_engine(n_params, n_workers, lr, momentum, c_beta, variant, workspace_dev, workspace_bytes, true);
}

void ga_destroy(ga_engine* e) {
    if (!e) return;
    DeviceGuard guard(e->device);
    cudaStreamSynchronize(e->stream);
    if (e->owns_state) {
        cudaFree(e->theta);
        cudaFree(e->vel);
        cudaFree(e->mom);
        cudaFree(e->saved);
        cudaFree(e->vworker);
        cudaFree(e->sec);
        cudaFree(e->partials);
        cudaFree(e->stats_dev);
    }
    free_layers(e);
    cudaFreeHost(e->pull_err);
    for (int s = 0; s < kHostStages; ++s) {
        cudaFree(e->stage[s]);
        if (e->ev_h2d[s]) cudaEventDestroy(e->ev_h2d[s]);
        if (e->ev_kernel[s]) cudaEventDestroy(e->ev_kernel[s]);
    }
    if (e->ev_prev) cudaEventDestroy(e->ev_prev);
    for (int q = 0; q < kHostD2hRing; ++q) if (e->ev_d2h[q]) cudaEventDestroy(e->ev_d2h[q]);
    if (e->s_h2d) cudaStreamDestroy(e->s_h2d);
    if (e->s_d2h) cudaStreamDestroy(e->s_d2h);
    cudaGetLastError();
    delete e;
}

int ga_set_stream(ga_engine* e, void* cuda_stream) {
    if (int rc = check_engine(e)) return rc;
    cudaStream_t next = (cudaStream_t)cuda_stream;
    if (next != e->stream) {
        // what the engine already enqueued on the old stream comes before anything it enqueues on
        // the new one: every launch reads the state the launch before it wrote
        DeviceGuard guard(e->device);
        cudaEvent_t done = nullptr;
        GA_CUDA(e, cudaEventCreateWithFlags(&done, cudaEventDisableTiming));
        cudaError_t err = cudaEventRecord(done, e->stream);
        if (err == cudaSuccess) err = cudaStreamWaitEvent(next, done, 0);
        cudaEventDestroy(done);   // released once the record has completed
        GA_CUDA(e, err);
        e->stream = next;
    }
    return GA_OK;
}

int ga_set_lr(ga_engine* e, float lr) {
    if (int rc = check_engine(e)) return rc;
    if (!(lr > 0.f) || !std::isfinite(lr)) return fail(GA_ERR_ARG, "lr must be positive and finite");
    e->lr = lr;
    return GA_OK;
}

int ga_set_layers(ga_engine* e, const int64_t* offsets_host, int n_layers) {
    if (int rc = check_engine(e)) return rc;
    if (!e->is_layer()) return fail(GA_ERR_STATE, "only the GA_GA_LAYER variant has layers");
    if (e->k_done != 0) return fail(GA_ERR_STATE, "layers can only be set before the first arrival");
    if (!offsets_host || n_layers < 1 || n_layers > (1 << 20)) return fail(GA_ERR_ARG, "bad layer table");
    if (offsets_host[0] != 0 || offsets_host[n_layers] != e->d)
        return fail(GA_ERR_ARG, "layer offsets must start at 0 and end at n_params");
    for (int p = 0; p < n_layers; ++p)
        if (offsets_host[p + 1] <= offsets_host[p]) return fail(GA_ERR_ARG, "layer %d is empty or out of order", p);
    DeviceGuard guard(e->device);
    if (int rc = sync_and_check(e)) return rc;
    return build_layers(e, offsets_host, n_layers);
}

int ga_num_layers(ga_engine* e) {
    if (int rc = check_engine(e)) return rc;
    if (!e->is_layer()) return fail(GA_ERR_STATE, "only the GA_GA_LAYER variant has layers");
    return e->n_layers();
}

int ga_get_layer_state(ga_engine* e, float* gaps_host, float* m_host) {
    if (int rc = check_engine(e)) return rc;
    if (!e->is_layer()) return fail(GA_ERR_STATE, "only the GA_GA_LAYER variant has layers");
    DeviceGuard guard(e->device);
    const size_t bytes = sizeof(float) * e->n_layers();
    if (gaps_host) GA_CUDA(e, cudaMemcpyAsync(gaps_host, e->layer_gap, bytes, cudaMemcpyDeviceToHost, e->stream));
    if (m_host) GA_CUDA(e, cudaMemcpyAsync(m_host, e->m_layer, bytes, cudaMemcpyDeviceToHost, e->stream));
    return sync_and_check(e);
}

int ga_set_params(ga_engine* e, const float* theta0_dev) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_dev_ptr(e, theta0_dev, "theta0_dev")) return rc;
    DeviceGuard guard(e->device);
    ga::ga_set_params_kernel<<<grid_1d(e->stride, 256, e->sms * 8), 256, 0, e->stream>>>(
        theta0_dev, e->theta, e->vel, e->mom, e->saved, e->vworker, e->n_workers, e->d, e->stride);
    GA_CUDA(e, cudaGetLastError());
    if (e->sec) GA_CUDA(e, cudaMemsetAsync(e->sec, 0, sizeof(float) * (size_t)e->stride, e->stream));
    if (e->m_layer) GA_CUDA(e, cudaMemsetAsync(e->m_layer, 0, sizeof(float) * e->n_layers(), e->stream));
    std::fill(e->iter.begin(), e->iter.end(), 0);
    e->k_done = 0;
    e->k_c = 0;
    e->stats_total = 0;
    return GA_OK;
}

const float* ga_pull(ga_engine* e, int worker) {
    if (check_engine(e) || check_worker(e, worker)) return nullptr;
    DeviceGuard guard(e->device);
    if (e->is_dana()) {   // the worker is sent the look-ahead estimate, not theta
        ga::ga_pull_estimate_kernel<<<grid_1d(e->stride, 256, e->sms * 8), 256, 0, e->stream>>>(
            e->theta, e->vel, e->hyper().eta_gamma, e->stride, e->row(worker));
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) { cuda_fail(e, err, "ga_pull launch"); return nullptr; }
        e->iter[worker] = e->k_done;
        return e->row(worker);
    }
    const long long bytes = e->stride * (long long)sizeof(float);
    const long long chunks = (bytes + ga::kPullChunk - 1) / ga::kPullChunk;
    const long long max_grid = (long long)e->sms * ga::kPullBlocksPerSm;
    const int grid = (int)(chunks < max_grid ? chunks : max_grid);
    ga::ga_pull_bulk_kernel<<<grid, 32, ga::kPullStages * ga::kPullChunk, e->stream>>>(
        e->theta, e->row(worker), bytes, e->pull_err);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { cuda_fail(e, err, "ga_pull launch"); return nullptr; }
    e->iter[worker] = e->k_done;
    return e->row(worker);
}

const float* ga_saved(ga_engine* e, int worker) {
    if (check_engine(e) || check_worker(e, worker)) return nullptr;
    return e->row(worker);
}

int64_t ga_push(ga_engine* e, int worker, const float* grad_dev) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_worker(e, worker)) return rc;
    if (int rc = check_dev_ptr(e, grad_dev, "grad_dev")) return rc;
    DeviceGuard guard(e->device);
    ga::Window w;
    int64_t tau = 0;
    e->stats_total = 0;
    fill_window(e, w, &worker, &grad_dev, 1, /*with_pull=*/false, &tau);
    if (e->is_layer()) {
        if (int rc = launch_layer_arrivals(e, w, false, nullptr, 0.f)) return rc;
        return tau;
    }
    if (int rc = launch_window(e, w, 0, e->stride / 4, e->stream)) return rc;
    return tau;
}

int ga_push_batch(ga_engine* e, const int* schedule_host, const float* const* grads_host, int K,
                  int64_t* delays_out_host) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = validate_batch(e, schedule_host, (const void* const*)grads_host, K, true)) return rc;
    DeviceGuard guard(e->device);
    int launches = 0;
    if (K > 0) e->stats_total = 0;
    if (e->is_layer()) {
        // A layer's norm needs the whole layer between arrivals, so they are not fused in time the way
        // the parameter-wise kernel fuses them: one launch per arrival after a distance pass, chained
        // so that each overlaps the tail of the one before (ga_layer_kernels.cuh). A worker may repeat
        // freely; the table is filled 16 arrivals at a time.
        ga::Window cur, nxt;
        int n_cur = K < ga::kMaxWindow ? K : ga::kMaxWindow;
        if (K > 0) fill_window(e, cur, schedule_host, grads_host, n_cur, true, delays_out_host);
        for (int pos = 0; pos < K;) {
            const int after = pos + n_cur;
            const int n_nxt = K - after < ga::kMaxWindow ? K - after : ga::kMaxWindow;
            if (n_nxt > 0)
                fill_window(e, nxt, schedule_host + after, grads_host + after, n_nxt, true,
                            delays_out_host ? delays_out_host + after : nullptr);
            if (int rc = launch_layer_arrivals(e, cur, pos > 0, n_nxt > 0 ? nxt.saved[0] : nullptr,
                                               n_nxt > 0 ? nxt.inv_bias[0] : 0.f))
                return rc;
            launches += n_cur + (pos == 0 ? 1 : 0);
            pos = after;
            cur = nxt;
            n_cur = n_nxt;
        }
        return launches;
    }
    for (int pos = 0; pos < K;) {
        const int n = next_window(schedule_host, pos, K, e->window);
        ga::Window w;
        fill_window(e, w, schedule_host + pos, grads_host + pos, n, true,
                    delays_out_host ? delays_out_host + pos : nullptr);
        if (int rc = launch_window(e, w, 0, e->stride / 4, e->stream)) return rc;
        ++launches;
        pos += n;
    }
    return launches;
}

int ga_push_batch_host(ga_engine* e, const int* schedule_host, const float* const* grads_host, int K,
                       int64_t* delays_out_host, float* const* sent_out_host) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = validate_batch(e, schedule_host, (const void* const*)grads_host, K, false)) return rc;
    if (sent_out_host)
        for (int j = 0; j < K; ++j)
            if (!sent_out_host[j]) return fail(GA_ERR_ARG, "sent_out_host[%d] is NULL", j);
    // a device pointer where host memory is expected would make the copies fail half-way through the
    // call: refuse it up front (the copies are whole vectors, so one query per buffer costs nothing)
    for (int j = 0; j < K; ++j) {
        for (const void* p : {(const void*)grads_host[j], (const void*)(sent_out_host ? sent_out_host[j] : nullptr)}) {
            cudaPointerAttributes attr;
            if (!p) continue;
            if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) { cudaGetLastError(); continue; }
            if (attr.type == cudaMemoryTypeDevice)
                return fail(GA_ERR_ARG, "buffer %d of ga_push_batch_host is device memory; use ga_push_batch", j);
        }
    }
    DeviceGuard guard(e->device);
    if (int rc = ensure_host_path(e)) return rc;
    int launches = 0;
    if (K > 0) e->stats_total = 0;
    if (e->is_layer()) {
        // Whole gradients, kLayerHostGroup arrivals at a time: copies-in of group g+1 and copies-out
        // of group g-1 run beside the launches of group g (one distance pass + one launch per
        // arrival). A group ends where a worker would repeat, so every sent copy is read out before
        // it is written again. Small groups keep the call's first copy-in and last copy-out, which
        // nothing overlaps, short.
        GA_CUDA(e, cudaEventRecord(e->ev_prev, e->stream));
        GA_CUDA(e, cudaStreamWaitEvent(e->s_h2d, e->ev_prev, 0));
        GA_CUDA(e, cudaStreamWaitEvent(e->s_d2h, e->ev_prev, 0));
        const int group = e->window < kLayerHostGroup ? e->window : kLayerHostGroup;
        const size_t vec_bytes = sizeof(float) * (size_t)e->d;
        long long g = 0;
        for (int pos = 0; pos < K; ++g) {
            const int n = next_window(schedule_host, pos, K, group);
            const int s = (int)(g % kHostStages);
            if (g >= kHostStages) GA_CUDA(e, cudaStreamWaitEvent(e->s_h2d, e->ev_kernel[s], 0));
            const float* staged[ga::kMaxWindow] = {};
            for (int j = 0; j < n; ++j) {
                float* dst = e->stage[s] + (size_t)j * e->stride;
                GA_CUDA(e, cudaMemcpyAsync(dst, grads_host[pos + j], vec_bytes, cudaMemcpyHostToDevice, e->s_h2d));
                staged[j] = dst;
            }
            GA_CUDA(e, cudaEventRecord(e->ev_h2d[s], e->s_h2d));
            GA_CUDA(e, cudaStreamWaitEvent(e->stream, e->ev_h2d[s], 0));
            // the copies out of the group before this one read saved rows that this group may rewrite
            if (sent_out_host && g >= 1) GA_CUDA(e, cudaStreamWaitEvent(e->stream, e->ev_d2h[(g - 1) % kHostD2hRing], 0));
            ga::Window w;
            fill_window(e, w, schedule_host + pos, staged, n, true, delays_out_host ? delays_out_host + pos : nullptr);
            if (int rc = launch_layer_arrivals(e, w, false, nullptr, 0.f)) return rc;
            launches += n + 1;
            GA_CUDA(e, cudaEventRecord(e->ev_kernel[s], e->stream));
            if (sent_out_host) {
                GA_CUDA(e, cudaStreamWaitEvent(e->s_d2h, e->ev_kernel[s], 0));
                for (int j = 0; j < n; ++j)
                    GA_CUDA(e, cudaMemcpyAsync(sent_out_host[pos + j], e->row(schedule_host[pos + j]), vec_bytes,
                                               cudaMemcpyDeviceToHost, e->s_d2h));
                GA_CUDA(e, cudaEventRecord(e->ev_d2h[g % kHostD2hRing], e->s_d2h));
            }
            pos += n;
        }
        GA_CUDA(e, cudaStreamSynchronize(e->s_h2d));
        GA_CUDA(e, cudaStreamSynchronize(e->s_d2h));
        if (int rc = sync_and_check(e)) return rc;
        return launches;
    }
    const long long chunk = e->stage_elems;
    const long long n_chunks = (e->stride + chunk - 1) / chunk;
    // How far the update kernels may run ahead of the copies back to the host. The kernel of
    // window w+1 on chunk c may rewrite a saved row that the copy-out of (w, c) still reads; copies
    // out run in order on one stream, so waiting for the copy-out issued `lag` chunks ago covers it.
    const long long lag = n_chunks < kHostD2hRing ? n_chunks : kHostD2hRing;
    // the copy streams start after everything already enqueued on the engine's stream
    GA_CUDA(e, cudaEventRecord(e->ev_prev, e->stream));
    GA_CUDA(e, cudaStreamWaitEvent(e->s_h2d, e->ev_prev, 0));
    GA_CUDA(e, cudaStreamWaitEvent(e->s_d2h, e->ev_prev, 0));
    long long g = 0;   // chunks issued in this call, over all windows: nothing below waits on the host
    for (int pos = 0; pos < K;) {
        const int n = next_window(schedule_host, pos, K, e->window);
        ga::Window w;
        const float* staged[ga::kMaxWindow] = {};
        fill_window(e, w, schedule_host + pos, staged, n, true, delays_out_host ? delays_out_host + pos : nullptr);
        for (long long c0 = 0, c = 0; c0 < e->stride; c0 += chunk, ++c, ++g) {
            const int s = (int)(g % kHostStages);
            const long long c1 = c0 + chunk < e->stride ? c0 + chunk : e->stride;
            const long long valid = (c1 < e->d ? c1 : e->d) - c0;   // floats the caller's buffers hold
            // staging buffer s is free once the kernel that read it kHostStages chunks ago has run
            if (g >= kHostStages) GA_CUDA(e, cudaStreamWaitEvent(e->s_h2d, e->ev_kernel[s], 0));
            for (int j = 0; j < n; ++j) {
                float* dst = e->stage[s] + (size_t)j * chunk;
                if (valid > 0)
                    GA_CUDA(e, cudaMemcpyAsync(dst, grads_host[pos + j] + c0, sizeof(float) * (size_t)valid,
                                               cudaMemcpyHostToDevice, e->s_h2d));
                w.grad[j] = dst;
            }
            GA_CUDA(e, cudaEventRecord(e->ev_h2d[s], e->s_h2d));
            GA_CUDA(e, cudaStreamWaitEvent(e->stream, e->ev_h2d[s], 0));
            if (sent_out_host && g >= lag)
                GA_CUDA(e, cudaStreamWaitEvent(e->stream, e->ev_d2h[(g - lag) % kHostD2hRing], 0));
            w.grad_offset = c0;
            if (int rc = launch_window(e, w, c0 / 4, c1 / 4, e->stream, /*first_range=*/c == 0, /*last_range=*/c1 == e->stride))
                return rc;
            ++launches;
            GA_CUDA(e, cudaEventRecord(e->ev_kernel[s], e->stream));
            if (sent_out_host) {
                GA_CUDA(e, cudaStreamWaitEvent(e->s_d2h, e->ev_kernel[s], 0));
                for (int j = 0; j < n && valid > 0; ++j)
                    GA_CUDA(e, cudaMemcpyAsync(sent_out_host[pos + j] + c0, e->row(schedule_host[pos + j]) + c0,
                                               sizeof(float) * (size_t)valid, cudaMemcpyDeviceToHost, e->s_d2h));
                GA_CUDA(e, cudaEventRecord(e->ev_d2h[g % kHostD2hRing], e->s_d2h));
            }
        }
        pos += n;
    }
    GA_CUDA(e, cudaStreamSynchronize(e->s_h2d));
    GA_CUDA(e, cudaStreamSynchronize(e->s_d2h));
    if (int rc = sync_and_check(e)) return rc;
    return launches;
}

int ga_get(ga_engine* e, int which, float* out_dev) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_dev_ptr(e, out_dev, "out_dev")) return rc;
    DeviceGuard guard(e->device);
    const float* src = which == GA_THETA ? e->theta : which == GA_V ? e->vel : which == GA_M ? e->mom : nullptr;
    if (which == GA_V2) {
        if (!e->is_adam()) return fail(GA_ERR_STATE, "only the Adam variants keep a second moment");
        src = e->sec;
    }
    if (src) {
        GA_CUDA(e, cudaMemcpyAsync(out_dev, src, sizeof(float) * (size_t)e->d, cudaMemcpyDeviceToDevice, e->stream));
    } else if (which == GA_C && e->is_layer()) {
        return fail(GA_ERR_STATE, "the layer-wise variant has one C per layer: see ga_get_layer_state");
    } else if (which == GA_C) {
        ga::ga_coeff_kernel<<<grid_1d(e->d, 256, e->sms * 8), 256, 0, e->stream>>>(e->mom, e->inv_bias(e->k_c),
                                                                               e->hyper(), e->d, out_dev);
        GA_CUDA(e, cudaGetLastError());
    } else {
        return fail(GA_ERR_ARG, "unknown vector %d", which);
    }
    return sync_and_check(e);
}

int ga_get_worker_momentum(ga_engine* e, int worker, float* out_dev) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_worker(e, worker)) return rc;
    if (int rc = check_dev_ptr(e, out_dev, "out_dev")) return rc;
    if (!e->is_dana()) return fail(GA_ERR_STATE, "only the DANA variants keep a momentum vector per worker");
    DeviceGuard guard(e->device);
    GA_CUDA(e, cudaMemcpyAsync(out_dev, e->vrow(worker), sizeof(float) * (size_t)e->d, cudaMemcpyDeviceToDevice, e->stream));
    return sync_and_check(e);
}

int ga_gap(ga_engine* e, int worker, float* gap_out_dev) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_worker(e, worker)) return rc;
    if (int rc = check_dev_ptr(e, gap_out_dev, "gap_out_dev")) return rc;
    if (e->is_layer()) return fail(GA_ERR_STATE, "the layer-wise variant has one Gap per layer: see ga_get_layer_state");
    DeviceGuard guard(e->device);
    ga::ga_gap_kernel<<<grid_1d(e->d, 256, e->sms * 8), 256, 0, e->stream>>>(
        e->theta, e->row(worker), e->mom, e->inv_bias(e->k_c), e->hyper(), e->d, gap_out_dev);
    GA_CUDA(e, cudaGetLastError());
    return sync_and_check(e);
}

int ga_set_option(ga_engine* e, int key, double value) {
    if (int rc = check_engine(e)) return rc;
    const int v = (int)value;
    switch (key) {
        case GA_OPT_C_ORDER:
            if (v != 0 && v != 1) return fail(GA_ERR_ARG, "GA_OPT_C_ORDER must be 0 or 1");
            if (v == 1 && e->is_layer()) return fail(GA_ERR_STATE, "the layer-wise Gap has the lagged order only");
            if (e->k_done != 0) return fail(GA_ERR_STATE, "GA_OPT_C_ORDER can only change before the first arrival");
            e->c_order = v;
            return GA_OK;
        case GA_OPT_MATH:
            if (v != 0 && v != 1) return fail(GA_ERR_ARG, "GA_OPT_MATH must be 0 or 1");
            e->fast_math = v;
            return GA_OK;
        case GA_OPT_STATS:
            if (v != 0 && v != 1) return fail(GA_ERR_ARG, "GA_OPT_STATS must be 0 or 1");
            e->stats = v;
            if (!v) e->stats_total = 0;
            return GA_OK;
        case GA_OPT_ADAM_BETA2:
            if (!(value >= 0.0 && value < 1.0)) return fail(GA_ERR_ARG, "GA_OPT_ADAM_BETA2 must be in [0, 1)");
            if (e->k_done != 0) return fail(GA_ERR_STATE, "GA_OPT_ADAM_BETA2 can only change before the first arrival");
            e->beta2 = (float)value;
            return GA_OK;
        case GA_OPT_ADAM_EPS:
            if (!((float)value > 0.f) || !std::isfinite((float)value))
                return fail(GA_ERR_ARG, "GA_OPT_ADAM_EPS must be positive and finite as a float");
            if (e->k_done != 0) return fail(GA_ERR_STATE, "GA_OPT_ADAM_EPS can only change before the first arrival");
            e->adam_eps = (float)value;
            return GA_OK;
        case GA_OPT_NESTEROV:
            if (v != 0 && v != 1) return fail(GA_ERR_ARG, "GA_OPT_NESTEROV must be 0 or 1");
            if (v && (e->is_dana() || e->is_adam()))
                return fail(GA_ERR_STATE, "the Nesterov step exists for the one-momentum-vector variants only");
            e->nesterov = v;
            return GA_OK;
        case GA_OPT_WEIGHT_DECAY:
            if (!(value >= 0.0) || !std::isfinite(value)) return fail(GA_ERR_ARG, "GA_OPT_WEIGHT_DECAY must be >= 0");
            e->weight_decay = (float)value;
            return GA_OK;
        case GA_OPT_WINDOW:
            if (v < 1 || v > GA_MAX_WINDOW) return fail(GA_ERR_ARG, "GA_OPT_WINDOW must be in [1, %d]", GA_MAX_WINDOW);
            e->window = v;
            return GA_OK;
        default:
            return fail(GA_ERR_ARG, "unknown option %d", key);
    }
}

int ga_get_stats_window(ga_engine* e, double* sum_gap_host, double* max_gap_host, int cap) {
    if (int rc = check_engine(e)) return rc;
    if (cap < 0 || (cap > 0 && (!sum_gap_host || !max_gap_host))) return fail(GA_ERR_ARG, "bad output arrays");
    if (!e->stats || !e->is_gap() || e->is_layer())
        return fail(GA_ERR_STATE, "no Gap statistics: set GA_OPT_STATS on a parameter-wise Gap-Aware variant first");
    const int64_t kept = e->stats_total < kStatsLog ? e->stats_total : kStatsLog;
    const int n = (int)(kept < cap ? kept : cap);
    if (n == 0) return 0;
    DeviceGuard guard(e->device);
    std::vector<double> host(2 * (size_t)kStatsLog);
    GA_CUDA(e, cudaMemcpyAsync(host.data(), e->stats_dev, sizeof(double) * host.size(), cudaMemcpyDeviceToHost, e->stream));
    if (int rc = sync_and_check(e)) return rc;
    for (int q = 0; q < n; ++q) {
        const int64_t slot = (e->stats_total - n + q) % kStatsLog;
        sum_gap_host[q] = host[2 * slot];
        max_gap_host[q] = host[2 * slot + 1];
    }
    return n;
}

int ga_get_stats(ga_engine* e, double* sum_gap, double* max_gap) {
    if (int rc = check_engine(e)) return rc;
    if (!sum_gap || !max_gap) return fail(GA_ERR_ARG, "output pointer is NULL");
    if (e->stats_total == 0) return fail(GA_ERR_STATE, "no Gap statistics: enable GA_OPT_STATS before a GA push");
    const int n = ga_get_stats_window(e, sum_gap, max_gap, 1);
    return n == 1 ? GA_OK : (n < 0 ? n : fail(GA_ERR_STATE, "no Gap statistics available"));
}

int64_t ga_num_arrivals(ga_engine* e) {
    if (int rc = check_engine(e)) return rc;
    return e->k_done;
}

int64_t ga_worker_iter(ga_engine* e, int worker) {
    if (int rc = check_engine(e)) return rc;
    if (int rc = check_worker(e, worker)) return rc;
    return e->iter[worker];
}

// ---- checkpoint layout: header, iter[n_workers], theta[d], v[d], m[d], saved[n_workers][d]
struct StateHeader {
    uint32_t magic, version;
    int64_t d, n_workers, k_done, k_c;
    float lr, gamma, beta, eps;
    int32_t variant, c_order, fast_math, stats, window, nesterov;
    float beta2, adam_eps, lr_max, weight_decay;
};

size_t ga_export_state(ga_engine* e, void* buf_host, size_t cap) {
    if (check_engine(e)) return 0;
    const size_t vec = sizeof(float) * (size_t)e->d;
    const size_t rows = 3 + (size_t)e->n_workers * (e->is_dana() ? 2 : 1) + (e->is_adam() ? 1 : 0);
    const size_t layer_bytes = e->is_layer() ? sizeof(int64_t) * (e->n_layers() + 2) + sizeof(float) * e->n_layers() : 0;
    const size_t need = sizeof(StateHeader) + sizeof(int64_t) * e->n_workers + vec * rows + layer_bytes;
    if (!buf_host || cap < need) return need;
    DeviceGuard guard(e->device);
    StateHeader h{};
    h.magic = kStateMagic; h.version = 2;
    h.beta2 = e->beta2; h.adam_eps = e->adam_eps; h.lr_max = e->lr_max; h.weight_decay = e->weight_decay;
    h.d = e->d; h.n_workers = e->n_workers; h.k_done = e->k_done; h.k_c = e->k_c;
    h.lr = e->lr; h.gamma = e->gamma; h.beta = e->beta; h.eps = e->eps;
    h.variant = e->variant; h.c_order = e->c_order; h.fast_math = e->fast_math; h.stats = e->stats; h.window = e->window; h.nesterov = e->nesterov;
    char* p = (char*)buf_host;
    std::memcpy(p, &h, sizeof h); p += sizeof h;
    std::memcpy(p, e->iter.data(), sizeof(int64_t) * e->n_workers); p += sizeof(int64_t) * e->n_workers;
    const float* vecs[3] = {e->theta, e->vel, e->mom};
    cudaError_t err = cudaSuccess;
    for (int q = 0; q < 3 && err == cudaSuccess; ++q, p += vec)
        err = cudaMemcpyAsync(p, vecs[q], vec, cudaMemcpyDeviceToHost, e->stream);
    for (int i = 0; i < e->n_workers && err == cudaSuccess; ++i, p += vec)
        err = cudaMemcpyAsync(p, e->row(i), vec, cudaMemcpyDeviceToHost, e->stream);
    for (int i = 0; e->is_dana() && i < e->n_workers && err == cudaSuccess; ++i, p += vec)
        err = cudaMemcpyAsync(p, e->vrow(i), vec, cudaMemcpyDeviceToHost, e->stream);
    if (e->is_adam() && err == cudaSuccess) { err = cudaMemcpyAsync(p, e->sec, vec, cudaMemcpyDeviceToHost, e->stream); p += vec; }
    if (e->is_layer() && err == cudaSuccess) {   // n_layers, offsets[n+1], m_p[n]
        const int64_t n = e->n_layers();
        std::memcpy(p, &n, sizeof n); p += sizeof n;
        std::memcpy(p, e->layer_off.data(), sizeof(int64_t) * (n + 1)); p += sizeof(int64_t) * (n + 1);
        err = cudaMemcpyAsync(p, e->m_layer, sizeof(float) * n, cudaMemcpyDeviceToHost, e->stream);
    }
    if (err != cudaSuccess) { cuda_fail(e, err, "ga_export_state"); return 0; }
    if (sync_and_check(e) != GA_OK) return 0;
    return need;
}

int ga_import_state(ga_engine* e, const void* buf_host, size_t len) {
    if (int rc = check_engine(e)) return rc;
    if (!buf_host || len < sizeof(StateHeader)) return fail(GA_ERR_ARG, "state buffer too short");
    StateHeader h;
    std::memcpy(&h, buf_host, sizeof h);
    if (h.magic != kStateMagic || h.version != 2) return fail(GA_ERR_ARG, "not a state written by ga_export_state");
    if (h.d != e->d || h.n_workers != e->n_workers)
        return fail(GA_ERR_ARG, "state is for %lld parameters / %lld workers", (long long)h.d, (long long)h.n_workers);
    const size_t vec = sizeof(float) * (size_t)e->d;
    if (h.variant != e->variant) return fail(GA_ERR_ARG, "state is for variant %d, engine is variant %d", h.variant, e->variant);
    const size_t rows = 3 + (size_t)e->n_workers * (e->is_dana() ? 2 : 1) + (e->is_adam() ? 1 : 0);
    const size_t layer_bytes = e->is_layer() ? sizeof(int64_t) * (e->n_layers() + 2) + sizeof(float) * e->n_layers() : 0;
    const size_t need = sizeof(StateHeader) + sizeof(int64_t) * e->n_workers + vec * rows + layer_bytes;
    if (e->is_layer()) {   // the layer table decides the true length
        const size_t base = sizeof(StateHeader) + sizeof(int64_t) * e->n_workers + vec * rows;
        if (len < base + sizeof(int64_t)) return fail(GA_ERR_ARG, "state buffer truncated");
        int64_t n = 0;
        std::memcpy(&n, (const char*)buf_host + base, sizeof n);
        if (n < 1 || n > (1 << 20) || len < base + sizeof(int64_t) * (n + 2) + sizeof(float) * n)
            return fail(GA_ERR_ARG, "state buffer truncated");
    } else if (len < need) return fail(GA_ERR_ARG, "state buffer truncated");
    // everything a later push relies on is checked before any device state is touched
    auto flag = [](int32_t v) { return v == 0 || v == 1; };
    auto unit = [](float v) { return v >= 0.f && v < 1.f; };
    if (h.window < 1 || h.window > GA_MAX_WINDOW || h.k_done < 0 || h.k_c < 0 || h.k_c > h.k_done ||
        !flag(h.c_order) || !flag(h.fast_math) || !flag(h.stats) || !flag(h.nesterov) ||
        !(h.lr > 0.f) || !std::isfinite(h.lr) || !(h.lr_max > 0.f) || !std::isfinite(h.lr_max) ||
        !(h.lr_max * h.eps > 0.f) || !(h.eps > 0.f) || !std::isfinite(h.eps) || !(std::fabs(h.gamma) < 1.f) ||
        !unit(h.beta) || !unit(h.beta2) || !(h.adam_eps > 0.f) || !std::isfinite(h.adam_eps) ||
        !(h.weight_decay >= 0.f) || !std::isfinite(h.weight_decay) ||
        (h.c_order == 1 && e->is_layer()) || (h.nesterov == 1 && (e->is_dana() || e->is_adam())))
        return fail(GA_ERR_ARG, "state header holds invalid values");
    const char* p = (const char*)buf_host + sizeof h;
    std::vector<int64_t> iter(e->n_workers);
    std::memcpy(iter.data(), p, sizeof(int64_t) * e->n_workers); p += sizeof(int64_t) * e->n_workers;
    for (int i = 0; i < e->n_workers; ++i)   // a pull cannot lie in the future: every delay stays >= 1
        if (iter[i] < 0 || iter[i] > h.k_done)
            return fail(GA_ERR_ARG, "state holds iter[%d] = %lld outside [0, %lld]", i, (long long)iter[i], (long long)h.k_done);
    // The second moments are running averages of squares. A negative entry could never arise and
    // would reach a square root; the kernels' short forms rely on its absence.
    {
        const char* base = (const char*)buf_host + sizeof(StateHeader) + sizeof(int64_t) * e->n_workers;
        auto has_negative = [&](size_t row) {
            const float* v = (const float*)(base + vec * row);
            for (long long j = 0; j < e->d; ++j) if (v[j] < 0.f) return true;
            return false;
        };
        const size_t adam_row = 3 + (size_t)e->n_workers * (e->is_dana() ? 2 : 1);
        if (has_negative(2) || (e->is_adam() && has_negative(adam_row)))
            return fail(GA_ERR_ARG, "state holds a negative second moment");
    }
    if (e->is_layer()) {   // the layer table too, before anything is copied
        const char* q = (const char*)buf_host + sizeof(StateHeader) + sizeof(int64_t) * e->n_workers + vec * rows;
        int64_t n = 0;
        std::memcpy(&n, q, sizeof n); q += sizeof n;
        std::vector<int64_t> off(n + 1);
        std::memcpy(off.data(), q, sizeof(int64_t) * (n + 1));
        if (off[0] != 0 || off[n] != e->d) return fail(GA_ERR_ARG, "state holds a layer table for another vector");
        for (int64_t t = 0; t < n; ++t) if (off[t + 1] <= off[t]) return fail(GA_ERR_ARG, "state holds a bad layer table");
    }
    DeviceGuard guard(e->device);
    float* vecs[3] = {e->theta, e->vel, e->mom};
    for (int q = 0; q < 3; ++q, p += vec)
        GA_CUDA(e, cudaMemcpyAsync(vecs[q], p, vec, cudaMemcpyHostToDevice, e->stream));
    for (int i = 0; i < e->n_workers; ++i, p += vec)
        GA_CUDA(e, cudaMemcpyAsync(e->row(i), p, vec, cudaMemcpyHostToDevice, e->stream));
    for (int i = 0; e->is_dana() && i < e->n_workers; ++i, p += vec)
        GA_CUDA(e, cudaMemcpyAsync(e->vrow(i), p, vec, cudaMemcpyHostToDevice, e->stream));
    if (e->is_adam()) { GA_CUDA(e, cudaMemcpyAsync(e->sec, p, vec, cudaMemcpyHostToDevice, e->stream)); p += vec; }
    if (e->is_layer()) {
        int64_t n = 0;
        std::memcpy(&n, p, sizeof n); p += sizeof n;
        std::vector<int64_t> off(n + 1);
        std::memcpy(off.data(), p, sizeof(int64_t) * (n + 1)); p += sizeof(int64_t) * (n + 1);
        if (int rc = build_layers(e, off.data(), (int)n)) return rc;
        GA_CUDA(e, cudaMemcpyAsync(e->m_layer, p, sizeof(float) * n, cudaMemcpyHostToDevice, e->stream));
    }
    if (int rc = sync_and_check(e)) return rc;
    e->iter = iter;
    e->k_done = h.k_done; e->k_c = h.k_c;
    e->lr = h.lr; e->gamma = h.gamma; e->beta = h.beta; e->eps = h.eps;
    e->beta2 = h.beta2; e->adam_eps = h.adam_eps; e->lr_max = h.lr_max; e->weight_decay = h.weight_decay;
    e->c_order = h.c_order; e->fast_math = h.fast_math; e->stats = h.stats; e->window = h.window; e->nesterov = h.nesterov;
    e->stats_total = 0;
    return GA_OK;
}

}  // extern "C"

// ============================================================ self-test of the short exact forms
extern "C" int64_t ga_selftest_exact_forms(int level, void* cuda_stream) {
    if (level < 0 || level > 1) return fail(GA_ERR_ARG, "level must be 0 or 1");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    unsigned long long* bad = nullptr;
    if (cudaMalloc(&bad, 2 * sizeof *bad) != cudaSuccess) { cudaGetLastError(); return fail(GA_ERR_OOM, "cannot allocate the counters"); }
    auto done = [&](int64_t rc) { cudaFree(bad); return rc; };
    if (cudaMemsetAsync(bad, 0, 2 * sizeof *bad, st) != cudaSuccess) return done(fail(GA_ERR_CUDA, "cudaMemsetAsync failed"));
    namespace t = ga::selftest;
    const int grid = 148 * 16, block = 256;
    t::rcp_range<<<grid, block, 0, st>>>(0x0d800000u, 0x71800001u, bad);                 // every b in [2^-100, 2^100]
    t::sqrt_range<<<grid, block, 0, st>>>(0x0d800000u, 0x7f800000u, 1e-8f, bad);          // every x in [2^-100, FLT_MAX]
    t::div_window<<<grid, block, 0, st>>>(-100, 100, -100, 100, -124, 126, 1u << 13, 1, bad);   // 2 x 3.3e8 pairs
    t::div_window<<<grid, block, 0, st>>>(-101, 127, -76, 105, -25, 100, 1u << 13, 2, bad);     // dist / C
    t::div_window<<<grid, block, 0, st>>>(-60, 127, -27, 65, -124, 100, 1u << 14, 3, bad);      // Adam's step
    for (float c : {0.1f, 0.01f, 1.0f, 0.001f, 0.5f}) t::div_const<<<grid, block, 0, st>>>(c, bad);
    t::gap_small_dist<<<grid, block, 0, st>>>(1u << 19, 4, bad);
    t::div_by_delay<<<grid, block, 0, st>>>(16, 5, bad);                                          // Adam-SA's g / tau
    if (level >= 1)
        for (uint32_t slice = 0; slice < 64; ++slice) t::div_all_significands<<<1024, 128, 0, st>>>(slice << 17, bad);
    // the comparison itself is checked too: beyond 2^126 the short reciprocal is known to differ from
    // the IEEE one (its result would be subnormal), so the second counter must come back non-zero
    t::rcp_range<<<4, block, 0, st>>>(0x7e800000u, 0x7e800400u, bad + 1);
    unsigned long long host[2] = {0, 0};
    cudaError_t err = cudaGetLastError();
    if (err == cudaSuccess) err = cudaMemcpyAsync(host, bad, sizeof host, cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess) err = cudaStreamSynchronize(st);
    if (err != cudaSuccess) return done(fail(GA_ERR_CUDA, "ga_selftest_exact_forms: %s", cudaGetErrorString(err)));
    if (host[1] == 0) return done(fail(GA_ERR_STATE, "the self-test did not see a difference where one is known to exist"));
    return done((int64_t)host[0]);
}

// A wait inside the layer-wise kernels that nothing satisfies: it has to give up and say so.
extern "C" int ga_selftest_bounded_wait(ga_engine* engine, void* cuda_stream) {
    if (engine && engine->cuda_failed) return fail(GA_ERR_CUDA, "engine is unusable after an earlier CUDA error");
    cudaStream_t st = engine ? engine->stream : (cudaStream_t)cuda_stream;
    unsigned int* epoch = nullptr;   // epoch word, then the abort word
    int* gave_up = nullptr;
    int* own_flag = nullptr;         // mapped host memory, like an engine's error flag
    int rc = GA_OK;
    if (cudaMalloc(&epoch, 2 * sizeof *epoch) != cudaSuccess || cudaMalloc(&gave_up, sizeof *gave_up) != cudaSuccess ||
        (!engine && cudaHostAlloc(&own_flag, sizeof *own_flag, cudaHostAllocMapped) != cudaSuccess)) {
        cudaGetLastError();
        rc = fail(GA_ERR_OOM, "cannot allocate the probe's words");
    } else {
        int* flag = engine ? engine->pull_err : own_flag;   // an engine's own flag: its next synchronising call reports it
        if (!engine) *flag = 0;
        int host_gave_up = -1;
        cudaError_t err = cudaMemsetAsync(epoch, 0, 2 * sizeof *epoch, st);
        if (err == cudaSuccess) err = cudaMemsetAsync(gave_up, 0xff, sizeof *gave_up, st);
        if (err == cudaSuccess) {
            ga::ga_layer_wait_probe_kernel<<<1, ga::kLayerThreads, 0, st>>>(epoch, (int*)(epoch + 1), flag, gave_up);
            err = cudaGetLastError();
        }
        if (err == cudaSuccess) err = cudaMemcpyAsync(&host_gave_up, gave_up, sizeof host_gave_up, cudaMemcpyDeviceToHost, st);
        if (err == cudaSuccess) err = cudaStreamSynchronize(st);
        if (err != cudaSuccess) rc = fail(GA_ERR_CUDA, "ga_selftest_bounded_wait: %s", cudaGetErrorString(err));
        else if (host_gave_up != 1 || *(volatile int*)flag != 2)
            rc = fail(GA_ERR_STATE, "the wait did not give up as it should (gave_up %d, flag %d)", host_gave_up, *flag);
    }
    cudaFree(epoch);
    cudaFree(gave_up);
    if (own_flag) cudaFreeHost(own_flag);
    return rc;
}

// ============================================================ allocation-free Gap statistics
// Everything this entry point needs lives in this file: the scratch array is part of the
// library's device image, so no call here ever allocates or frees device memory.
namespace {

constexpr int kNoAllocTile = 4096;          // parameters reduced by one block
constexpr int kNoAllocMaxBlocks = (int)(GA_NOALLOC_MAX_PARAMS / kNoAllocTile);   // 65536
constexpr int kNoAllocMaxDevices = 64;

// One partial result per block. In host code this name is only a handle for
// cudaGetSymbolAddress; kernels are given the address that call returns.
static __device__ __align__(256) ga::StatsPartial g_noalloc_partials[kNoAllocMaxBlocks];

// First pass: block b reduces parameters [b*4096, (b+1)*4096) and overwrites partials[b].
__global__ void __launch_bounds__(256)
ga_gap_stats_tile_kernel(const float* __restrict__ theta, const float* __restrict__ saved,
                         const float* __restrict__ mom, float inv_bias, ga::Hyper h, long long d,
                         ga::StatsPartial* __restrict__ partials) {
    __shared__ double s_sum[8];
    __shared__ float s_max[8];
    const long long tile = (long long)blockIdx.x * kNoAllocTile;
    double sum = 0.0;
    float mx = 0.f;
    for (int q = 0; q < kNoAllocTile / (256 * 4); ++q) {
        const long long e = tile + ((long long)q * 256 + threadIdx.x) * 4;
        float t[4], s[4], m[4];
        int n = 0;
        if (e + 4 <= d) {
            const float4 a = *reinterpret_cast<const float4*>(theta + e);
            const float4 b = *reinterpret_cast<const float4*>(saved + e);
            const float4 c = *reinterpret_cast<const float4*>(mom + e);
            t[0] = a.x; t[1] = a.y; t[2] = a.z; t[3] = a.w;
            s[0] = b.x; s[1] = b.y; s[2] = b.z; s[3] = b.w;
            m[0] = c.x; m[1] = c.y; m[2] = c.z; m[3] = c.w;
            n = 4;
        } else {
            for (; n < 4 && e + n < d; ++n) { t[n] = theta[e + n]; s[n] = saved[e + n]; m[n] = mom[e + n]; }
        }
        for (int u = 0; u < n; ++u) {
            const float C = __fmul_rn(h.eta_max, __fadd_rn(__fsqrt_rn(__fmul_rn(m[u], inv_bias)), h.eps));
            const float G = __fadd_rn(__fdiv_rn(fabsf(__fsub_rn(t[u], s[u])), C), 1.0f);
            sum += (double)G;
            mx = fmaxf(mx, G);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sum += __shfl_xor_sync(0xffffffffu, sum, o);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if ((threadIdx.x & 31) == 0) { s_sum[threadIdx.x >> 5] = sum; s_max[threadIdx.x >> 5] = mx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        ga::StatsPartial out;
        out.sum = 0.0; out.max = 0.f; out.pad = 0.f;
        for (int w = 0; w < 8; ++w) { out.sum += s_sum[w]; out.max = fmaxf(out.max, s_max[w]); }
        partials[blockIdx.x] = out;
    }
}

// Device address of the scratch array, looked up once per device.
ga::StatsPartial* g_noalloc_addr[kNoAllocMaxDevices] = {};

int noalloc_scratch(ga::StatsPartial** out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return fail(GA_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(err));
    if (dev < 0 || dev >= kNoAllocMaxDevices) return fail(GA_ERR_ARG, "device index %d not supported", dev);
    ga::StatsPartial* p = __atomic_load_n(&g_noalloc_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        err = cudaGetSymbolAddress((void**)&p, g_noalloc_partials);   // the current device's copy
        if (err != cudaSuccess || !p)
            return fail(GA_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(err));
        __atomic_store_n(&g_noalloc_addr[dev], p, __ATOMIC_RELEASE);
    }
    *out = p;
    return GA_OK;
}

}  // namespace

extern "C" int ga_gap_stats_noalloc(const float* theta_dev, const float* saved_dev, const float* m_dev,
                                    size_t n_params, float lr_max, float c_beta, int64_t n_refreshes,
                                    double* out_dev, void* cuda_stream) {
    if (int rc = check_dev_ptr(theta_dev, "theta_dev")) return rc;
    if (int rc = check_dev_ptr(saved_dev, "saved_dev")) return rc;
    if (int rc = check_dev_ptr(m_dev, "m_dev")) return rc;
    if (!out_dev || (uintptr_t)out_dev % 8) return fail(GA_ERR_ARG, "out_dev is NULL or not 8-byte aligned");
    if (n_params == 0) return fail(GA_ERR_ARG, "n_params is 0");
    if (n_params > GA_NOALLOC_MAX_PARAMS)
        return fail(GA_ERR_ARG, "n_params = %zu exceeds GA_NOALLOC_MAX_PARAMS = %zu, the size the fixed scratch array covers",
                    n_params, (size_t)GA_NOALLOC_MAX_PARAMS);
    if (!(lr_max > 0.f) || !std::isfinite(lr_max)) return fail(GA_ERR_ARG, "lr_max must be positive and finite");
    if (!(c_beta >= 0.f && c_beta < 1.f)) return fail(GA_ERR_ARG, "c_beta must be in [0, 1)");
    if (n_refreshes < 0) return fail(GA_ERR_ARG, "n_refreshes is negative");
    ga::StatsPartial* scratch = nullptr;
    if (int rc = noalloc_scratch(&scratch)) return rc;
    ga::Hyper h;
    h = ga::Hyper{};
    h.eta_max = lr_max; h.beta = c_beta; h.one_minus_beta = (float)(1.0 - (double)c_beta); h.eps = 1e-8f;
    const float inv_bias = n_refreshes == 0 ? 0.f : (float)(1.0 / (1.0 - std::pow((double)c_beta, (double)n_refreshes)));
    const int blocks = (int)((n_params + kNoAllocTile - 1) / kNoAllocTile);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    ga_gap_stats_tile_kernel<<<blocks, 256, 0, st>>>(theta_dev, saved_dev, m_dev, inv_bias, h, (long long)n_params, scratch);
    ga::ga_stats_finish_kernel<<<1, 256, 0, st>>>(scratch, blocks, out_dev, 0, 1, 0);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return fail(GA_ERR_CUDA, "ga_gap_stats_noalloc launch: %s", cudaGetErrorString(err));
    return GA_OK;
}
