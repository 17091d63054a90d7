/* fdg -- one training iteration of a network split into K modules under fully decoupled parallel
 * backpropagation, combined with N data-parallel workers whose stale gradients are averaged
 * before an SGD update.  C ABI of the sm_100a library (libfdg.so).
 *
 * What one call of fdg_step computes (paper Sec. 3.2, Sec. 3.3, Eq. "dl_update", Algorithm 1),
 * with k = 1..K the module, t = 0,1,... the iteration, M = n_workers * per_worker_batch:
 *   - module k runs its layers forward on the batch sampled at  tau_f = t - k + 1  (if >= 0)
 *     with its current weights w_k(t), reading what module k-1 produced in iteration t-1;
 *   - module k back-propagates the batch  tau_b = t - 2K + k + 1  (if >= 0) using the error
 *     gradient module k+1 produced in iteration t-1, the activations it stashed when it
 *     forwarded that batch, and the weights it had then, w_k(t - 2K + 2k);
 *   - every worker's gradient is the sum over its per_worker_batch samples scaled by
 *     1/per_worker_batch; the workers are mixed by P = (1/N) 1 1^T, i.e. averaged, so that
 *     w_k(t+1) = w_k(t) - lr * mean over all M samples of dphi/dw_k; the average is taken inside
 *     the weight-gradient contraction, which reduces over the worker x batch axis;
 *   - while tau_b < 0 the gradient is zero and w_k(t+1) = w_k(t).
 * phi is softmax cross-entropy (natural logarithm).  Batch-norm uses the statistics of each
 * worker's own per_worker_batch * H * W values (biased variance, eps = 1e-5).
 *
 * Conventions
 *   - Every function returns an fdg_status; nothing aborts or throws; on error, outputs are
 *     left untouched and fdg_last_error() describes the failure.
 *   - "device" pointers are CUDA device pointers on the context's device, "host" pointers are
 *     ordinary host memory.  The caller owns every buffer it passes; the context owns all
 *     device memory it obtained through the allocator and releases it in fdg_destroy.
 *   - Activations are NHWC, worker-major: rows s*B .. (s+1)*B-1 belong to worker s.
 *   - Canonical parameter order: layers in list order; per layer W then b (linear W[out][in];
 *     conv W[c_out][kh][kw][c_in]); batch-norm gamma then beta; a projecting FDG_RES_ADD
 *     carries Wp[c_out][c_in], gamma_p, beta_p.
 *   - The library needs an sm_100 device; there is no CPU path.
 *   - Threads: calls on one context must not overlap in time; different contexts are independent.  Everything a
 *     call enqueues runs asynchronously on the context's streams.
 */
#ifndef FDG_H
#define FDG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define FDG_API __attribute__((visibility("default")))
#else
#define FDG_API
#endif

typedef struct fdg_ctx fdg_ctx;          /* opaque; owns all device state */

typedef enum {
    FDG_OK = 0,
    FDG_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, unknown enum value          */
    FDG_ERR_BAD_SPLIT = 2,     /* split points not strictly increasing / cut a residual block  */
    FDG_ERR_UNSUPPORTED = 3,   /* a shape the kernels do not cover (e.g. odd size before pool) */
    FDG_ERR_ARCH = 4,          /* no CUDA device of compute capability 10.x                    */
    FDG_ERR_OOM = 5,           /* the allocator returned NULL                                  */
    FDG_ERR_CUDA = 6,          /* a CUDA runtime call failed (message in fdg_last_error)       */
    FDG_ERR_TIMEOUT = 7,       /* a bounded device-side wait gave up                           */
    FDG_ERR_STATE = 8          /* call order violated (e.g. step before set_params)            */
} fdg_status;

typedef enum {
    FDG_LINEAR = 0,            /* y = x W^T + b over the flattened sample                       */
    FDG_CONV3X3 = 1,           /* padding 1, stride 1 or 2                                      */
    FDG_CONV1X1 = 2,           /* padding 0, stride 1 or 2                                      */
    FDG_RELU = 3,
    FDG_MAXPOOL2 = 4,          /* 2x2 window, stride 2; ties: first maximum in row-major order  */
    FDG_GLOBAL_AVGPOOL = 5,
    FDG_BATCHNORM = 6,         /* per-worker batch statistics                                   */
    FDG_RES_BEGIN = 7,         /* remember the current tensor as the shortcut                   */
    FDG_RES_ADD = 8            /* add the shortcut (flags & 1: through conv1x1(stride) + BN)    */
} fdg_layer_kind;

/* flags: bit 0 = has bias (LINEAR / CONV*), or "projection shortcut" (RES_ADD). */
typedef struct { int32_t kind, c_in, c_out, stride, flags; } fdg_layer;

/* Device-memory allocator of the caller (e.g. PyTorch's caching allocator).  alloc returns a
 * device pointer aligned to at least 256 bytes or NULL; free receives what alloc returned. */
typedef struct {
    void* (*alloc)(size_t bytes, void* user);
    void  (*free)(void* ptr, void* user);
    void* user;
} fdg_allocator;

typedef struct {
    int32_t dtype;             /* 0: fp32 everywhere.  1: bf16 activations / weight copies /
                                  error gradients, fp32 accumulation, fp32 master weights       */
    int32_t in_h, in_w, in_c;  /* sample shape; 1,1,3072 for an MLP on flattened 32x32x3 inputs */
    int32_t num_classes;       /* must equal the last layer's c_out                             */
    int32_t serial;            /* 1: run every module on one stream (results are bit-identical
                                  to the concurrent mode when both contexts have the same
                                  grid_sms; used to test the event wiring)                      */
    int32_t kernel_path;       /* 0: tensor-core kernels where shapes allow (bf16 only), the 256-column
                                     tile (and the 128-column tile of 3x3 stride-1 layers on 16x16 images) as
                                     pairs of CTAs on two SMs (tcgen05 cta_group::2);
                                  1: plain FMA kernels only;
                                  2: tensor-core kernels, no CTA pairs (bit-identical results to 0 wherever
                                     both run the same loop order: everything but those 128-column layers) */
    int32_t worker_groups;     /* 0 or 1: every kernel covers all workers.  n > 1: every module but the last runs
                                  its layers once per group of n_workers / n workers (n rounded down to a power
                                  of two that divides n_workers; ignored where a group would cut a tensor-core
                                  tile) and adds the groups' parameter gradients; results differ from n = 1 only
                                  in fp32 summation order.  Smaller launches, more of them: measured slower on a
                                  B200 at every n for the ResNet-18-shaped benchmark, so it is off by default     */
    void* const* streams;      /* K cudaStream_t of the caller (one per module, for its backward pass and update),
                                  or NULL: the library creates them                                             */
    const double* mixing;      /* NULL: P = (1/N) 1 1^T, the exact average; every worker then holds the same weights and
                                  the library keeps ONE copy per module and takes the average inside the
                                  weight-gradient contraction.
                                  Otherwise: host array, N x N row-major, the weight matrix P of Sec. 2.3 (Eq.
                                  "weight_matrix": P_ij = alpha on the edges of the model-group graph, 1 - kappa_i alpha on
                                  the diagonal); every row must sum to 1.  The library then keeps one weight replica
                                  w^_{s,k} per worker s and module k, runs every layer once per worker on that
                                  worker's replica (plain FMA kernels: kernel_path is taken as 1), computes each
                                  worker's own gradient with scale 1/per_worker_batch, and updates
                                  u_{s,k} = w^_{s,k} - lr g_{s,k},  w^_{s,k}(t+1) = sum_r P_sr u_{r,k}  (Eq. "dl_update").
                                  At most 32 workers.  The matrix is copied.                                     */
    int32_t grid_sms;          /* SMs the persistent kernels (tensor-core convolutions / GEMMs, streamed batch-norm) size
                                  their grids for.  0: a third of the device's SMs when the modules run on streams of their
                                  own (the concurrency of Sec. 3.2: a tensor-core kernel of one module then runs beside a
                                  memory-bound kernel of another instead of after it), all of them with serial = 1.
                                  n > 0: n SMs (clamped to the device).  Results depend on it only through fp32 summation
                                  order (contraction splits, batch-norm row chunks): two contexts with the same value are
                                  bit-identical whatever their streams                                              */
} fdg_options;

/* Stash policy.  Every activation a module's backward pass needs is kept from the module's forward pass of
 * that batch (iteration tau+k-1) until its backward pass (iteration tau+2K-k-1): "store all", the h~_k(tau) of
 * Sec. 3.2.  There is no recompute-from-module-input mode: the largest configuration this library is run on
 * (ResNet-18-shaped, K = 8, 16 workers x 256) holds its whole stash in the 180 GB of one B200, and
 * fdg_create fails with FDG_ERR_OOM before any launch when the allocator cannot supply it.
 *
 * Build a context.  Paper: the split of layers 1..L into groups g(1)..g(K) (Sec. 3.2) and the
 * S x K agents of Sec. 3.3, all placed on the current CUDA device.
 *   layers/n_layers : the network, host array.
 *   split_points    : host array of K-1 layer indices (0-based): first layer of modules 2..K.
 *   n_workers, per_worker_batch : N and B; every step consumes M = N*B samples.
 *   lr              : step size eta (changeable later with fdg_set_lr).
 *   alloc           : NULL selects cudaMalloc/cudaFree.
 * Fails with BAD_SPLIT / UNSUPPORTED / ARCH / OOM before any kernel is launched. */
FDG_API fdg_status fdg_create(const fdg_layer* layers, int32_t n_layers,
                      const int32_t* split_points, int32_t K,
                      int32_t n_workers, int32_t per_worker_batch, float lr,
                      const fdg_options* opt, const fdg_allocator* alloc, fdg_ctx** out);

/* The SM count the context's persistent kernels are sized for (fdg_options.grid_sms after the automatic choice). */
FDG_API fdg_status fdg_grid_sms(const fdg_ctx* ctx, int32_t* sms);

/* Number of parameters (length of the canonical parameter vector). */
FDG_API fdg_status fdg_param_count(const fdg_ctx* ctx, size_t* count);

/* Where every tensor sits in the canonical parameter vector (the order fdg_set_params, fdg_params and fdg_grads
 * use): one record per tensor, in that order.  Paper: the per-layer weights w_l of Sec. 2.1 grouped into the modules
 * g(k) = {p_k .. q_k} of Sec. 3.2.
 *   layer  : index into the layer list given to fdg_create
 *   module : k - 1 of the module that owns the layer
 *   role   : FDG_PARAM_W (linear [out][in]; conv [c_out][kh][kw][c_in]), _BIAS, _GAMMA, _BETA, and for a projecting
 *            FDG_RES_ADD  _PROJ_W [c_out][1][1][c_in], _PROJ_GAMMA, _PROJ_BETA
 *   ndim, shape[4] : extents, outermost first (unused trailing extents are 1)
 *   offset, count  : first element and number of elements in the canonical vector
 * out may be NULL to query the number of tensors; otherwise at most `capacity` records are written and *count
 * receives the total number. */
typedef enum { FDG_PARAM_W = 0, FDG_PARAM_BIAS = 1, FDG_PARAM_GAMMA = 2, FDG_PARAM_BETA = 3,
               FDG_PARAM_PROJ_W = 4, FDG_PARAM_PROJ_GAMMA = 5, FDG_PARAM_PROJ_BETA = 6 } fdg_param_role;
typedef struct { int32_t layer, module, role, ndim; int64_t shape[4]; uint64_t offset, count; } fdg_param_tensor;
FDG_API fdg_status fdg_param_layout(const fdg_ctx* ctx, fdg_param_tensor* out, int32_t capacity, int32_t* count);

/* Load version-0 weights from a host fp32 array in canonical order (the library draws no random
 * numbers).  Resets the iteration counter to 0 and empties every FIFO. */
FDG_API fdg_status fdg_set_params(fdg_ctx* ctx, const float* host_params, size_t count);

/* Contexts created with a mixing matrix only: replace replica `worker` of the initial weights (after fdg_set_params,
 * before the first step), so that a run can start from replicas that differ (consensus error delta(0) > 0). */
FDG_API fdg_status fdg_set_params_worker(fdg_ctx* ctx, int32_t worker, const float* host_params, size_t count);

/* One iteration t of Algorithm 1 for all modules and workers (steps listed at the top).
 *   dev_inputs : device, [M, in_h, in_w, in_c] in the context's dtype (fp32 or bf16), the
 *                batch sampled at iteration t.  Its contents must be complete before the call
 *                (the library's streams do not synchronise with the caller's), and the buffer
 *                must stay valid and unchanged until the library has copied it into its own FIFO:
 *                that copy is enqueued on module 1's stream; fdg_wait_ingest() blocks until it
 *                is done.  The library does not keep the pointer.
 *   dev_labels : device, int32 [M].
 *   host_loss_or_null : if non-NULL the call waits until the last module has computed the loss
 *                of the batch it forwards in this iteration (tau = t-K+1; NaN while tau < 0) and
 *                stores its mean; the rest of the iteration (backward passes, updates) is still
 *                in flight when the call returns.  If NULL the call only enqueues work. */
FDG_API fdg_status fdg_step(fdg_ctx* ctx, const void* dev_inputs, const int32_t* dev_labels,
                    float* host_loss_or_null);

/* Same as fdg_step with HOST input buffers (pinned memory makes the copies asynchronous); the
 * host-to-device copies go straight into the FIFO slot, ordered on module 1's stream. */
FDG_API fdg_status fdg_step_host(fdg_ctx* ctx, const void* host_inputs, const int32_t* host_labels,
                         float* host_loss_or_null);

/* Block the host until the input/label copies of the most recent step have executed; after
 * that the caller may overwrite or free the buffers it passed to that step. */
FDG_API fdg_status fdg_wait_ingest(fdg_ctx* ctx);

/* Make `stream` (a cudaStream_t of the caller, NULL = the default stream) wait for everything the steps enqueued
 * so far: work the caller puts on that stream afterwards (an event record for timing, a kernel that reads the
 * caller's own buffers) runs after the last module's update of the most recent step.  Only enqueues waits. */
FDG_API fdg_status fdg_join(fdg_ctx* ctx, void* stream);

/* Wait for all modules, then copy the fp32 master weights w(t) (t = number of steps done) to a
 * host array in canonical order.  count receives the number of floats written.  Paper: the agents'
 * weights w^_{s,k}(t) of Eq. "dl_update" (b); with P = (1/N) 1 1^T and equal initial values they are the same
 * for every worker s (the consensus error of Sec. 4 is identically zero), so one copy is kept and returned. */
FDG_API fdg_status fdg_params(fdg_ctx* ctx, float* host_out, size_t capacity, size_t* count);

/* Debug twin of fdg_params: the gradients that entered the last step's update, i.e. the mean over the workers of
 * the stale gradients of Eq. "dl_update", (1/N) sum_s grad^_{w_{s,k}} Phi_s(t - 2K + k + 1) with the per-sample scale
 * 1/per_worker_batch (zeros for modules that had no backward batch yet: the gradient is 0 while tau < 0). */
FDG_API fdg_status fdg_grads(fdg_ctx* ctx, float* host_out, size_t capacity, size_t* count);

/* The weights w^_{s,k}(t) / the gradient g_{s,k} of ONE worker s.  Without a mixing matrix every worker has the same
 * weights (fdg_params_worker returns them for any s) and only the averaged gradient exists (fdg_grads_worker fails with
 * FDG_ERR_STATE).  With a mixing matrix fdg_params returns worker 0's weights and fdg_grads the mean over the workers. */
FDG_API fdg_status fdg_params_worker(fdg_ctx* ctx, int32_t worker, float* host_out, size_t capacity, size_t* count);
FDG_API fdg_status fdg_grads_worker(fdg_ctx* ctx, int32_t worker, float* host_out, size_t capacity, size_t* count);

/* Maximum consensus error of Sec. 5 (Eq. "max_consensus_error"):
 *   delta(t) = max over layers l and workers s of || w_{s,l}(t) - (1/N) sum_r w_{r,l}(t) ||_2
 * (a layer's tensors -- W with b, gamma with beta, a projection's three tensors -- form one vector w_{s,l}).  Waits for
 * the modules and evaluates the definition on the host in double precision.  0 without a mixing matrix. */
FDG_API fdg_status fdg_consensus_error(fdg_ctx* ctx, double* delta);

/* The delay schedule of Sec. 3.2 (forward batch t-k+1, backward batch t-2K+k+1, backward weights of version
 * t-2K+2k) as observed on the device in the last step.  Every FIFO slot carries a tag (batch id, weight version) in
 * device memory.  One small kernel per module and step, on the module's backward / update stream and ordered like the
 * step's other work by the neighbour events, first stamps the slots this step fills, then copies the tags of the
 * slots the step reads into a trace.  The trace therefore proves the slot arithmetic (which slot holds which batch and
 * version at which step); that the DATA in a slot is complete when it is read is what the event wiring guarantees
 * and the parity tests (and the bit-identity of the one-stream and the concurrent mode) check.
 * Arrays of K int64 (host):
 *   fwd_batch[k]          batch id found in the activation slot module k forwarded (-1 idle)
 *   bwd_batch[k]          batch id found in the stash slot module k back-propagated (-1 idle);
 *                         -2 if the error-gradient slot carried a different batch id
 *   bwd_weight_version[k] version tag of the weight slot the backward pass read (-1 idle) */
FDG_API fdg_status fdg_trace(fdg_ctx* ctx, int64_t* fwd_batch, int64_t* bwd_batch,
                     int64_t* bwd_weight_version, int32_t K);

/* Change the step size used by the following steps (a sequence eta_t, Algorithm 1's input). */
FDG_API fdg_status fdg_set_lr(fdg_ctx* ctx, float lr);

/* Bytes of device memory the context holds, and how many kernels it has launched so far. */
FDG_API fdg_status fdg_stats(const fdg_ctx* ctx, size_t* device_bytes, uint64_t* kernel_launches);

/* Device time of the last completed step of every module (ms, CUDA events on the module's
 * stream; array of K floats) -- waits for the modules. */
FDG_API fdg_status fdg_module_times(fdg_ctx* ctx, float* ms, int32_t K);

/* Per-kernel-class device timing for measurements.  fdg_profile(ctx, 1) clears the statistics and
 * makes every later launch record a CUDA event before and after itself on its own stream;
 * fdg_profile(ctx, 0) stops that.  fdg_profile_read waits for the device and returns one record
 * per kernel class that was launched: its launches, the summed event time (ms) and the summed
 * ALGORITHMIC flops and bytes of those launches, followed by records named "class[layer shape]"
 * that break the GEMM / convolution classes down by layer shape.  The statistics are process-wide. */
typedef struct { char name[48]; uint64_t launches; double ms, flops, bytes; } fdg_kernel_stat;
FDG_API fdg_status fdg_profile(fdg_ctx* ctx, int32_t enable);
FDG_API fdg_status fdg_profile_read(fdg_ctx* ctx, fdg_kernel_stat* out, int32_t capacity, int32_t* count);

/* Bias gradient without any allocation.  (The paper has no counterpart: this is a service entry
 * point, not a step of its method.)
 *
 * For whom: code that must not allocate device memory while it runs -- a plug-in living inside
 * another framework's memory pool, a latency-critical loop that forbids cudaMalloc/cudaFree because
 * they synchronise the whole device, a process whose memory budget was handed out up front.  Such a
 * caller cannot create an fdg_ctx (which allocates its FIFOs), yet may still need the reduction the
 * step uses for bias gradients:  dev_db[c] = sum over rows of dev_dy[row][c].
 *
 *   dev_dy  : device, [rows][channels] row-major, fp32 (dtype 0) or bf16 (dtype 1)
 *   dev_db  : device, fp32 [channels], overwritten
 *   stream  : a cudaStream_t (NULL = default stream); the call only enqueues two kernels
 * Limits and behaviour
 *   - channels <= FDG_STATIC_MAX_CHANNELS, rows >= 1; anything else returns FDG_ERR_INVALID_ARG and
 *     fdg_static_last_error() says why.  Nothing is launched in that case.
 *   - The partial sums go to a fixed 1 MiB array inside the library image (present on every GPU
 *     that loads the library, for the life of the process).  The entry point calls no cudaMalloc,
 *     cudaFree or any allocating routine.  The first call on a device may make the CUDA runtime load the
 *     library's device code (which is when the 1 MiB is reserved), so it doubles as the warm-up.
 *   - dev_dy, dev_db and the stream must belong to the CURRENT device: the array used is the current device's.
 *   - All calls on a device share that array.  It keeps the previous call's contents; nothing in it
 *     has to start at zero, because the first kernel writes every slot the second one reads.  Two
 *     calls that may overlap on the GPU (different streams, no ordering) race on it: order them.
 *   - The first call on each device looks the array's device address up (cudaGetSymbolAddress, with
 *     that device current).  Make that first call before starting any stream capture.
 *   - Same summation order on every call, so equal inputs give equal bits. */
#define FDG_STATIC_MAX_CHANNELS 4096
FDG_API fdg_status fdg_bias_grad_static(const void* dev_dy, int32_t dtype, int64_t rows, int32_t channels,
                                        float* dev_db, void* stream);
FDG_API const char* fdg_static_last_error(void);

FDG_API const char* fdg_last_error(const fdg_ctx* ctx);   /* ctx may be NULL: last create error */
FDG_API void        fdg_destroy(fdg_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FDG_H */
