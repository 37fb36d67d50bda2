/* ga.h -- C ABI of the Gap-Aware parameter-server ("master") update for NVIDIA B200.
 *
 * The library plays the master of asynchronous SGD with a parameter server
 * (arXiv 1909.10802, Section 4): it owns the master parameters theta, the momentum (update
 * vector) v, the running second moment m from which the coefficient C is derived, and one
 * saved copy of the parameters per worker (theta^i: what was last sent to worker i).
 * Each arriving gradient is applied by one fused CUDA kernel; several consecutive arrivals
 * can be applied by a single launch that keeps theta, v and m in registers.
 *
 * Conventions
 *   - fp32 throughout. Pointers named *_dev are DEVICE pointers, 16-byte aligned, to at least
 *     n_params floats; pointers named *_host are HOST pointers. The library owns theta, v, m
 *     and the saved copies (allocated in ga_create, freed in ga_destroy); the caller owns
 *     gradient buffers and every output buffer it passes in, and must keep a gradient buffer
 *     unchanged until the work enqueued by the call that reads it has finished. A *_dev pointer
 *     that the CUDA runtime reports as ordinary host memory, or as memory of a device that the
 *     engine's device cannot reach, is refused with GA_ERR_ARG before any kernel could touch it
 *     (asked once per pointer; pinned and managed memory pass). The length of a caller's buffer
 *     cannot be checked: a buffer shorter than n_params floats is the caller's error.
 *   - Work is enqueued on the stream bound with ga_set_stream (default: the legacy default
 *     stream) and the call returns after host bookkeeping; ga_get, ga_gap, ga_get_stats,
 *     ga_export_state and the *_host calls synchronise that stream before returning.
 *   - One engine serves one host thread at a time and lives on the device that was current
 *     when it was created.
 *   - No call aborts, traps or throws. Functions returning int give >= 0 on success or a
 *     negative GA_ERR_* code; ga_last_error() then describes the failure. A CUDA error is
 *     sticky: every later call on that engine returns GA_ERR_CUDA.
 *   - Delays: k counts arrivals from 1; iter[i] (initially 0) is the number of arrivals applied
 *     when worker i last pulled; the delay of an arrival is tau = k - iter[i] >= 1.
 */
#ifndef GA_H
#define GA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ga_engine ga_engine;

/* which master algorithm a push applies */
enum {
    GA_ASGD = 0, /* Algorithm "Momentum-ASGD: master" (Section 4)                      */
    GA_SA = 1,   /* Algorithm "Staleness-Aware: master" (Section 4.1): step eta / tau   */
    GA_GA = 2,   /* Algorithm "Gap-Aware: master" (Section 5), parameter-wise Gap (5.3) */
    GA_SA_GRAD = 3, /* Algorithm "Staleness-Aware-Gradient: master" (appendix): gradient / tau */
    /* The DANA masters (appendix, Algorithms "DANA: master", "DANA-Staleness-Aware: master",
     * "DANA-Gap-Aware: master"): one momentum vector v^i per worker; the master moves by
     * -eta v^i; a pull sends (and saves) the look-ahead estimate theta - eta gamma sum_j v^j.
     * The sum is kept as a running sum, (sum - old v^i) + new v^i. Costs one more N x n_params
     * array of device memory. */
    GA_DANA = 4,    /* v^i <- gamma v^i + g                                   */
    GA_DANA_SA = 5, /* v^i <- gamma v^i + g / tau                             */
    GA_DANA_GA = 6, /* v^i <- gamma v^i + (1/G) g, Gap against the saved estimate */
    /* The Adam masters (appendix, Algorithms "Adam: master", "Adam-Staleness-Aware: master",
     * "Adam-Gap-Aware: master"). `momentum` of ga_create is beta_1; beta_2 and Adam's epsilon are
     * options (defaults 0.999, 1e-8). The penalty enters the first moment only. For Adam-GA the
     * C algorithm is run with gamma = 0, i.e. on the raw gradient, with c_beta. */
    GA_ADAM = 7,    /* m <- beta1 m + (1-beta1) g                         */
    GA_ADAM_SA = 8, /* m <- beta1 m + (1-beta1) g / tau                   */
    GA_ADAM_GA = 9, /* m <- beta1 m + ((1-beta1)/G) g                     */
    /* Gap-Aware with the layer-wise Gap of Section 5.3: G_p = ||theta_p - theta^i_p|| / C_p + 1, one
     * number per layer (ga_set_layers); with a single layer -- the default -- it is the global Gap
     * of Definition 1. C_p comes from the C algorithm run on the squared norm of the layer's
     * update vector. Norms are accumulated in fp64 and rounded to fp32 once. A layer's norm must be
     * known before the layer is updated, so arrivals are not fused in time: each is one launch over
     * the vector, which inside a ga_push_batch call also measures the next arrival's distance (one
     * extra distance pass per call), and consecutive launches overlap. ga_push_batch_host stages
     * whole gradients for this variant (see there). */
    GA_GA_LAYER = 10
};

enum { GA_OK = 0, GA_ERR_ARG = -1, GA_ERR_STATE = -2, GA_ERR_OOM = -3, GA_ERR_CUDA = -4 };

/* vectors readable with ga_get; GA_V is the master's momentum v, sum_j v^j for the DANA variants,
 * Adam's first moment for the Adam variants; GA_V2 is Adam's second moment */
enum { GA_THETA = 0, GA_V = 1, GA_M = 2, GA_C = 3, GA_V2 = 4 };

/* options for ga_set_option */
enum {
    GA_OPT_C_ORDER = 0, /* 0 (default): the Gap of arrival k uses C as it stands after arrival
                           k-1, and m is then refreshed with the master's new v. 1: "Adam order":
                           m is first refreshed with (gamma v + g)^2 of the raw gradient (the
                           printed line of the C algorithm), then C, Gap and the step follow. */
    GA_OPT_MATH = 1,    /* 0 (default): exact -- every symbol of the algorithms is one IEEE
                           round-to-nearest operation, in their order (roots, divisions and reciprocals
                           by sequences that return the IEEE result: see ga_selftest_exact_forms).
                           1: fast: approximate reciprocal and square root, one division per
                           element (g*C/(|theta-theta^i|+C)); a few ulp off. Applies to GA_GA,
                           GA_DANA_GA and GA_ADAM_GA (there also to Adam's own root and division);
                           every other variant is always exact. On large vectors exact mode runs at
                           the memory roofline too, so fast mode buys nothing there. */
    GA_OPT_STATS = 2,   /* 1: every arrival of GA_GA, GA_DANA_GA and GA_ADAM_GA also reduces the sum
                           and the maximum of the Gap over all parameters (the average Gap is what
                           Appendix "Gap and Delay" logs); read with ga_get_stats_window or
                           ga_get_stats. Default 0. Not computed for GA_GA_LAYER, which has one Gap
                           per layer (see ga_get_layer_state). Non-finite values propagate by IEEE
                           rules and nothing traps; with this option on they are also noticed: the
                           sum of an arrival is NaN or infinite exactly when some parameter's Gap was. */
    GA_OPT_WINDOW = 3,  /* 1..16 (default 16): most arrivals fused into one launch by
                           ga_push_batch. */
    GA_OPT_ADAM_BETA2 = 4, /* Adam variants: beta_2 in [0,1), default 0.999; before the first arrival */
    GA_OPT_ADAM_EPS = 5,   /* Adam variants: epsilon > 0, default 1e-8; before the first arrival */
    GA_OPT_NESTEROV = 7,   /* 1: Nesterov form of the momentum step for GA_ASGD, GA_SA, GA_GA, GA_SA_GRAD and
                              GA_GA_LAYER: theta <- theta - eta (g_hat + gamma v_{k+1}) with g_hat the penalised
                              gradient. Section 6 says the experiments ran Nesterov momentum, but no
                              master algorithm is printed in that form; this is the form of the common
                              framework optimisers.
                              Default 0: the printed step theta - eta v_{k+1}. */
    GA_OPT_WEIGHT_DECAY = 6 /* lambda >= 0 (default 0): the master adds lambda * theta_k to every arriving
                              gradient before anything else, so the decay element is penalised with the
                              gradient (Appendix "Weight Decay") */
};

#define GA_MAX_WINDOW 16

/* Create a master for n_params parameters and n_workers workers. lr is eta (and eta_max of the
 * C algorithm), momentum is gamma (|gamma| < 1; Section 3, no dampening), c_beta is beta_1 of
 * Algorithm "C Coefficient Calculation" (0 <= c_beta < 1; the paper uses 0.999; eps is 1e-8).
 * All state starts at 0: theta = v = m = 0, every saved copy = 0, no arrivals, iter[] = 0.
 * lr must be large enough that lr * 1e-8, the smallest value C can take, does not round to zero
 * in fp32 (lr above about 1.5e-37). Returns NULL on invalid arguments or allocation failure (see
 * ga_last_error). */
ga_engine* ga_create(size_t n_params, int n_workers, float lr, float momentum, float c_beta,
                     int variant);

/* The same master inside memory the caller provides: for processes in which a framework's
 * allocator owns the device memory (the state of a master is large -- Appendix "Gap-Aware Overhead":
 * one copy of the parameters per worker -- and should then come out of that pool, not compete with
 * it). ga_workspace_bytes returns the size needed for theta, v, m, the n_workers saved copies, the
 * DANA variants' per-worker momentum vectors, Adam's second moment and the statistics buffers
 * (0 on invalid arguments); ga_create_in lays them out in workspace_dev (device memory, 256-byte
 * aligned, at least that many bytes, owned by the caller and kept alive and untouched until
 * ga_destroy, which does not free it). Everything else is as for ga_create. Still allocated by the
 * library itself: one word of pinned host memory per engine, the small per-layer tables of
 * GA_GA_LAYER (ga_set_layers) and the staging buffers of ga_push_batch_host on its first use. */
size_t ga_workspace_bytes(size_t n_params, int n_workers, int variant);
ga_engine* ga_create_in(size_t n_params, int n_workers, float lr, float momentum, float c_beta,
                        int variant, void* workspace_dev, size_t workspace_bytes);

/* Free everything the engine owns. NULL is accepted. Synchronises the bound stream first. */
void ga_destroy(ga_engine* e);

/* Enqueue all later work of this engine on cuda_stream (a cudaStream_t; NULL = default stream).
 * The new stream is made to wait (by an event) for the work this engine has already enqueued on
 * the stream it leaves, so a change of stream never reorders the engine's own launches. */
int ga_set_stream(ga_engine* e, void* cuda_stream);

/* Learning rate eta_k for the arrivals that follow (decay, warm-up: Appendix "Hyperparameters").
 * eta_max of the C algorithm stays the rate given to ga_create (Algorithm "C Coefficient
 * Calculation" takes the maximal rate as an input, normally the first one), so the Gap penalty
 * relaxes as the rate decays (Section 5.1). The momentum vector is kept free of the rate (v <- gamma
 * v + g_hat, theta <- theta - eta_k v, as the master algorithms are printed), so a change of rate
 * needs no correction of v. lr must be positive and finite. */
int ga_set_lr(ga_engine* e, float lr);

/* GA_GA_LAYER only, before the first arrival: layer p is elements [offsets_host[p],
 * offsets_host[p+1]); n_layers + 1 increasing offsets from 0 to n_params. Resets every m_p. */
int ga_set_layers(ga_engine* e, const int64_t* offsets_host, int n_layers);

/* GA_GA_LAYER only: the number of layers in force (1 until ga_set_layers or ga_import_state says
 * otherwise). Negative on error. */
int ga_num_layers(ga_engine* e);

/* GA_GA_LAYER only: the Gap G_p of every layer at the most recent arrival and the running second
 * moment m_p behind C_p, n_layers floats each, into host memory (either may be NULL). */
int ga_get_layer_state(ga_engine* e, float* gaps_host, float* m_host);

/* theta <- theta0 and every worker's saved copy <- theta0 (the initialisation step of Algorithm
 * "DANA-Gap-Aware: master"; the same convention is used for GA); v, m, the arrival counter and
 * iter[] are reset to 0. theta0_dev: n_params floats on the device. */
int ga_set_params(ga_engine* e, const float* theta0_dev);

/* The master's send step (the worker side of it is the first step of Algorithm "Momentum-ASGD:
 * worker"): copies the master parameters into worker's saved copy with TMA bulk copies (the DANA
 * variants compute and store the estimate theta - eta gamma sum_j v^j instead), records
 * iter[worker] <- arrivals applied so far, and returns the device address of that copy
 * (library-owned, stable for the engine's life; contents change at that worker's next pull or
 * batched push). NULL on error. */
const float* ga_pull(ga_engine* e, int worker);

/* Device address of worker's saved copy theta^worker (n_params floats) without copying anything:
 * the parameters that worker was last sent, from which it computes its next gradient
 * (Algorithm "Momentum-ASGD: worker"). Read-only for the caller. NULL on error. */
const float* ga_saved(ga_engine* e, int worker);

/* Apply one arriving gradient from `worker` (one iteration of the master algorithm of the
 * engine's variant, without the final "send"): delay, [C, Gap, penalised gradient], momentum,
 * step, [refresh of m]. grad_dev: n_params floats, unchanged until the work completes.
 * Returns the delay tau >= 1 of this arrival, or a negative error. A worker may push again
 * without pulling; its Gap is then still measured against its last saved copy. */
int64_t ga_push(ga_engine* e, int worker, const float* grad_dev);

/* K arrivals applied in the order given -- the master serves gradients first come, first served
 * (Appendix "Algorithms") -- each followed at once by that worker's pull, the save-and-send step
 * that closes Algorithm "Gap-Aware: master". Equivalent to { ga_push(schedule[j], grads[j]);
 * ga_pull(schedule[j]); } for j = 0..K-1, but up to GA_OPT_WINDOW consecutive arrivals are applied
 * by one kernel that reads and writes theta, v, m once (legal because every step is independent
 * per parameter, Section 5.3). A window is cut where a worker repeats. schedule_host: K worker
 * ids; grads_host: K device pointers (a HOST array of device pointers); delays_out_host: K delays,
 * may be NULL. K >= 0. Returns the number of kernel launches used, or a negative error (nothing
 * is applied on an argument error). */
int ga_push_batch(ga_engine* e, const int* schedule_host, const float* const* grads_host, int K,
                  int64_t* delays_out_host);

/* As ga_push_batch, for callers whose gradients and results live in HOST memory (pinned memory
 * gives full PCIe speed): grads_host[j] points to n_params floats on the host; when
 * sent_out_host is not NULL, sent_out_host[j] receives the parameters sent to worker
 * schedule[j] after its arrival (n_params floats each). The parameter range is processed in
 * chunks so that host-to-device copies, the update kernel and device-to-host copies overlap,
 * across the windows of the call as well as within them. Synchronous: returns when all results
 * are in host memory. Allocates its staging buffers (2 x 16 x 16 MiB) on first use. A buffer that
 * is device memory is refused (GA_ERR_ARG, nothing applied); pageable host memory works, slower.
 * GA_GA_LAYER needs a whole gradient before a layer's norm is known: there the call stages whole
 * vectors, one arrival at a time (two staging buffers of n_params floats), the copy-in of the next
 * arrival and the copy-out of the previous one running beside the launches of the current. */
int ga_push_batch_host(ga_engine* e, const int* schedule_host, const float* const* grads_host,
                       int K, int64_t* delays_out_host, float* const* sent_out_host);

/* Copy theta, v, m (which = GA_THETA, GA_V, GA_M) or the coefficient C derived from m as it
 * stands (GA_C; last two lines of the C algorithm) into out_dev (n_params floats). */
int ga_get(ga_engine* e, int which, float* out_dev);

/* DANA variants only: copy worker's momentum vector v^worker into out_dev (n_params floats).
 * GA_ERR_STATE for the other variants. */
int ga_get_worker_momentum(ga_engine* e, int worker, float* out_dev);

/* The parameter-wise Gap |theta - theta^worker| / C + 1 (Section 5.3) of `worker` against the
 * master as it stands, into gap_out_dev (n_params floats). Changes no state. */
int ga_gap(ga_engine* e, int worker, float* gap_out_dev);

int ga_set_option(ga_engine* e, int key, double value);

/* Gap statistics of every arrival of the most recent ga_push, ga_push_batch or
 * ga_push_batch_host call, oldest first: sum_gap_host[q] and max_gap_host[q] are the sum and the
 * maximum over all parameters of the Gap that arrival was penalised with (sum / n_params is the
 * average Gap that Appendix "Gap and Delay" logs; Section 5.1 compares it with the delay). All
 * windows of the call are covered, not only the last launch. Needs GA_OPT_STATS = 1 before the call
 * and a parameter-wise Gap-Aware variant (GA_GA, GA_DANA_GA, GA_ADAM_GA), else GA_ERR_STATE. The
 * engine keeps the last GA_STATS_LOG arrivals of a call; when the call had more, or cap is smaller,
 * the most recent ones are returned. Both arrays hold cap doubles on the host. The sum is
 * accumulated in fp64 in a fixed order (reproducible run to run). Synchronises the stream.
 * Returns the number of pairs written (0 when no arrival has been applied since the option was set,
 * ga_set_params or ga_import_state), or a negative error. */
#define GA_STATS_LOG 4096
int ga_get_stats_window(ga_engine* e, double* sum_gap_host, double* max_gap_host, int cap);

/* The last pair of ga_get_stats_window: the Gap statistics of the most recent arrival.
 * GA_ERR_STATE when none is available. */
int ga_get_stats(ga_engine* e, double* sum_gap, double* max_gap);

/* Arrivals applied so far, and iter[worker]. Negative on error. */
int64_t ga_num_arrivals(ga_engine* e);
int64_t ga_worker_iter(ga_engine* e, int worker);

/* Checkpoint: all state needed to continue bit-identically (hyper-parameters, options, counters,
 * iter[], theta, v, m, saved copies, and the workers' momentum vectors for DANA). ga_export_state returns the number of bytes needed; it
 * writes them when cap is large enough (buf_host may be NULL to query). ga_import_state needs an
 * engine created with the same n_params, n_workers and variant. */
size_t ga_export_state(ga_engine* e, void* buf_host, size_t cap);
int ga_import_state(ga_engine* e, const void* buf_host, size_t len);

/* Self-test of the kernels' exact arithmetic on the current device. In exact mode (GA_OPT_MATH = 0)
 * the Gap-Aware kernels evaluate the square root in C (Algorithm "C Coefficient Calculation"), the
 * division and the reciprocal of the Gap (Algorithm "Gap-Aware: master") and Adam's root and division
 * (Algorithm "Adam-Gap-Aware: master") by short sequences -- hardware seed, one Newton step, one
 * residual correction -- wherever the operands lie in ranges for which those sequences return
 * the IEEE round-to-nearest result, and by the general IEEE routines elsewhere. That claim rests on
 * the GPU's approximate reciprocal and reciprocal square root as well as on arithmetic, so this call
 * repeats the comparison with the IEEE routines on the device at hand:
 *   level 0 (well under a second): the reciprocal for every value in [2^-100, 2^100]; the square
 *     root for every value in [2^-100, FLT_MAX] and at 0; the division for 2 x 10^9 random significand
 *     pairs spread over every exponent pair of the windows the kernels use, for constant numerators
 *     over every divisor in [1, 2^100], and for tiny and subnormal distances;
 *   level 1 (about a minute): additionally the division for all 2^46 pairs of significands.
 * Returns the number of operands on which a short form differs from IEEE (0 on a B200), or a
 * negative GA_ERR_* code (GA_ERR_STATE if the comparison fails to see a difference planted outside
 * the ranges in use, where one is known to exist). Allocates 16 bytes of device memory for the
 * duration of the call and synchronises cuda_stream. */
int64_t ga_selftest_exact_forms(int level, void* cuda_stream);

/* Self-test of the bounded waits. The layer-wise kernels (GA_GA_LAYER) order consecutive arrivals by
 * waiting, layer by layer, for a counter that the previous arrival advances; like the bulk-copy waits
 * of ga_pull these waits have an iteration limit, after which the block raises the engine's error
 * flag and returns, and the engine reports GA_ERR_CUDA from its next synchronising call, for good.
 * This call launches one block that waits for a counter nothing advances and checks that the wait
 * runs out (after about a second), that the flag is raised and that the kernel returns, leaving the
 * context usable. With engine == NULL it uses a flag of its own on cuda_stream. With an engine it
 * raises THAT engine's flag (on the engine's stream; cuda_stream is ignored), which shows the whole
 * reporting path: the call itself returns GA_OK, and every later synchronising call on the engine
 * (ga_get, ga_get_stats, ...) returns GA_ERR_CUDA -- the engine is spent, as after a real lost wait.
 * Returns GA_OK, GA_ERR_STATE if the wait did not behave so, or another negative GA_ERR_* code.
 * Allocates a few words for the duration of the call; synchronises the stream. */
int ga_selftest_bounded_wait(ga_engine* engine, void* cuda_stream);

/* Gap statistics without any allocation. (The paper has no counterpart of this call; it exists
 * for deployment reasons only.) Computes the sum and the maximum over all parameters of the
 * parameter-wise Gap |theta - saved| / C + 1, with C = lr_max * (sqrt(m / (1 - c_beta^n_refreshes))
 * + 1e-8) (C = lr_max * 1e-8 when n_refreshes is 0) -- the same numbers ga_gap would give if its
 * output were reduced -- from three device vectors the caller already holds, and writes
 * out_dev[0] = sum, out_dev[1] = max (two doubles on the device).
 *
 * Who it is for: code that runs next to a training job whose framework allocator already owns
 * nearly all device memory (a raw cudaMalloc may then simply fail), and hooks on a latency-critical
 * path that must not pay the device-wide synchronisation that cudaMalloc and cudaFree imply. This
 * call needs no engine and never calls cudaMalloc, cudaFree or any allocating routine: the
 * per-block partial results of its reduction live in a fixed array inside the library's device
 * image (1 MiB, present on every GPU that loads the library until the process ends).
 *
 *   - theta_dev, saved_dev, m_dev: n_params floats each, device memory, 16-byte aligned, read only.
 *   - n_params must be in [1, GA_NOALLOC_MAX_PARAMS]; larger sizes are rejected with GA_ERR_ARG.
 *   - Work is enqueued on cuda_stream and the call returns at once; the result is in out_dev when
 *     that stream reaches this point.
 *   - The first call on each device looks up the device address of the fixed array (once per
 *     device, with that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array. Each call overwrites every entry it later reads,
 *     so nothing has to be cleared between calls, but two calls whose kernels overlap on the GPU
 *     (different streams, or different host threads) race on it: run them one after the other.
 * Returns GA_OK or a negative GA_ERR_* code (see ga_last_error). */
#define GA_NOALLOC_MAX_PARAMS ((size_t)1 << 28)
int ga_gap_stats_noalloc(const float* theta_dev, const float* saved_dev, const float* m_dev,
                         size_t n_params, float lr_max, float c_beta, int64_t n_refreshes,
                         double* out_dev, void* cuda_stream);

/* Message for the calling thread's most recent failure ("" if none). Never NULL. */
const char* ga_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* GA_H */
