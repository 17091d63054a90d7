// Internal launch interface between the step executor (fdg_api.cu) and the kernels.
// All pointers are device pointers; `dt` is 0 for fp32 storage, 1 for bf16 storage.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fdg {

struct ConvGeom {            // x: [N,H,W,C]  ->  y: [N,Ho,Wo,Co], R x R window
    int N, H, W, C, Ho, Wo, Co, R, stride, pad;
};

enum { EPI_RELU = 1, EPI_ACCUM = 2, EPI_OUT_F32 = 4 };

// Number of k-splits the weight-gradient kernel will use for this geometry (>= 1) and the
// fp32 workspace elements it needs (splits * Co * R*R*C when splits > 1, else 0).
int    wgrad_splits(const ConvGeom& g);
size_t wgrad_workspace_elems(const ConvGeom& g);

// y = conv(x, W) (+ bias) (relu)            (Eq. forward_step for linear / conv layers)
// workspace: forward_workspace_elems(g) floats (0: none needed), or nullptr: a forward pass with few output tiles and a
// long contraction is split over the contraction through it
size_t forward_workspace_elems(const ConvGeom& g);
void conv_forward(int dt, const void* x, const void* w, const float* bias, void* y, const ConvGeom& g,
                  int epi, float* workspace, size_t workspace_elems, cudaStream_t st);
// dx (+)= conv_transpose(dy, W)             (Eq. backward_step, gradient w.r.t. the layer input)
void conv_dgrad(int dt, const void* dy, const void* w, void* dx, const ConvGeom& g, int epi, cudaStream_t st);
// dW = sum over all N*Ho*Wo rows of dy^T (x) patches(x), fp32 out; the reduction runs over the
// worker x batch axis, which is the worker average of Eq. dl_update (b) for P = 11^T/N.
// accum: dw += (a second group of workers adds to the first group's result)
void conv_wgrad(int dt, const void* x, const void* dy, float* dw, float* workspace, const ConvGeom& g, bool accum, cudaStream_t st);
// db[c] = sum over rows of dy[row][c]; scratch: fp32 [64 * C]
void bias_grad(int dt, const void* dy, float* db, float* scratch, long rows, int C, bool accum, cudaStream_t st);

// Backward pass through "+ bias, ReLU" of a layer in one pass over dy: dy *= (y > 0) in place (y_or_null == nullptr: no
// ReLU) and db = column sums of the masked dy (db_or_null == nullptr: no bias).  scratch: relu_bias_backward_scratch_elems(C)
// floats.  Only for widths relu_bias_backward_supported() accepts.
bool   relu_bias_backward_supported(int dt, int C);
size_t relu_bias_backward_scratch_elems(int C);
void   relu_bias_backward(int dt, const void* y_or_null, void* dy, float* db_or_null, float* scratch, long rows, int C, bool accum, cudaStream_t st);

// First-layer convolution (3x3, stride 1, <= 4 input channels, bf16): dedicated kernels (stem.cu).
bool   stem_supported(int dt, const ConvGeom& g);
size_t stem_wgrad_workspace_elems(const ConvGeom& g);
void   stem_forward(const void* x, const void* w, const float* bias, void* y, const ConvGeom& g, bool relu, cudaStream_t st);
void   stem_wgrad(const void* x, const void* dy, float* dw, float* workspace, const ConvGeom& g, bool accum, cudaStream_t st);

void relu_forward(int dt, const void* x, void* y, size_t n, cudaStream_t st);
// dx (+)= dy * (y > 0)
void relu_backward(int dt, const void* y, const void* dy, void* dx, size_t n, bool accum, cudaStream_t st);
// y = a + b ; backward is two copies / accumulations
void add_forward(int dt, const void* a, const void* b, void* y, size_t n, cudaStream_t st);
void copy_or_accumulate(int dt, const void* src, void* dst, size_t n, bool accum, cudaStream_t st);
void maxpool_forward(int dt, const void* x, void* y, int N, int H, int W, int C, cudaStream_t st);
void maxpool_backward(int dt, const void* x, const void* dy, void* dx, int N, int H, int W, int C, bool accum, cudaStream_t st);
void gap_forward(int dt, const void* x, void* y, int N, int HW, int C, cudaStream_t st);
void gap_backward(int dt, const void* dy, void* dx, int N, int HW, int C, bool accum, cudaStream_t st);

// Batch-norm with per-worker statistics.  x: [n_workers * rows_per_worker, C].
// err: device word that a kernel sets non-zero if a bounded wait on an asynchronous copy gave up (nullptr: the
// kernels that stream through shared memory are not used).
// stats: fp32 [n_workers][C][2] = (mean, invstd).  scratch: fp32 [128 * n_workers * C * 2].
// conv_part / conv_chunks: if non-null, the producing convolution already left per-tile (sum, sum of squares)
// partials [n_workers * conv_chunks][C][2] (worker-major); the statistics pass over x is skipped.
// sms: the SMs the streamed kernels size their grids for (0 or >= the device's count: all); the partial sums depend on it
// through the number of row chunks (fp32 summation order).
void bn_forward(int dt, const void* x, const float* gamma, const float* beta, const void* residual_or_null,
                void* y, float* stats, float* scratch, int n_workers, long rows_per_worker, int C, bool relu,
                const float* conv_part, int conv_chunks, int sms, int* err, cudaStream_t st);
bool bn_accepts_conv_partials(int dt, int C);
// dy_eff = dout * (out > 0 if relu).  dx (+)= BN backward of dy_eff; dres (+)= dy_eff;
// dgamma, dbeta (fp32) = sums over all workers.  red: fp32 [n_workers][C][2] scratch for (sum dy, sum dy xhat).
void bn_backward(int dt, const void* x, const void* out, const void* dout, const float* gamma, const float* beta,
                 const float* stats, void* dx, bool accum_dx, void* dres_or_null, bool accum_dres, float* dgamma, float* dbeta,
                 float* red, float* scratch, int n_workers, long rows_per_worker, int C, bool relu, bool has_res, bool accum_params,
                 int sms, int* err, cudaStream_t st);

// Softmax cross-entropy over fp32 logits [M, classes]: dlogits (storage dtype) = (softmax - onehot) * scale,
// *loss_out = mean loss.  Deterministic single-block reduction.
void softmax_ce(int dt, const float* logits, const int32_t* labels, void* dlogits, float* loss_out, int M, int classes,
                float scale, cudaStream_t st);

// Classifier head (the last linear layer, c_in = K -> C classes, C <= 16) fused with the loss.  head_forward_loss: logits
// (fp32), dlogits = (softmax - onehot) * scale (storage dtype) and the mean loss in one launch; `counter` is a device word
// that is zero between launches.  head_backward: dx (+)= dlogits W (dx_or_null == nullptr: not needed), dW, db.
// scratch: head_scratch_elems floats, used by both (the loss partials follow the weight-gradient partials).
bool   head_supported(int dt, int K, int C);
size_t head_scratch_elems(int M, int K, int C);
void   head_forward_loss(int dt, const void* x, const void* W, const float* bias, const int32_t* labels, float* logits, void* dlogits, float* scratch,
                         unsigned* counter, float* loss_out, int M, int K, int C, float scale, cudaStream_t st);
void   head_backward(int dt, const void* x, const void* W, const void* dlogits, void* dx_or_null, bool accum_dx, float* dW, float* db_or_null, float* scratch,
                     int M, int K, int C, cudaStream_t st);

// master -= lr * grad (skipped when grad == nullptr: w(t+1) = w(t)); copy_next = storage-dtype copy of
// the new master (the next weight version).  n must be a multiple of 4; pointers 16-byte aligned.
void sgd_update(int dt, float* master, const float* grad, void* copy_next, size_t n, float lr, cudaStream_t st);

// General mixing matrix: R replicas [R][n_big + n_small] of master and grad; u_r = w_r - lr g_r (grad == nullptr: u_r = w_r),
// w_s = sum_r P[s][r] u_r in place, and the storage-dtype copies of the next version (replica r at copy0 + r * slot_bytes:
// n_big values of the storage dtype, then n_small floats).  R <= mix_max_replicas().
int  mix_max_replicas();
void mix_update(int dt, float* master, const float* grad, void* copy0, size_t n_big, size_t n_small, size_t slot_bytes, int R, const float* P, float lr,
                cudaStream_t st);

// Schedule tags (see fdg_trace).  tags are int64 pairs {batch id, weight version}.
struct TagOps {
    const int64_t* rd_act;  const int64_t* rd_stash; const int64_t* rd_grad; const int64_t* rd_wbwd; const int64_t* rd_wfwd;
    int64_t* wr_in; int64_t* wr_out; int64_t* wr_stash; int64_t* wr_grad; int64_t* wr_wnext;
    int64_t fwd_batch, bwd_batch, version_now;   // what this step produces (-1: nothing)
    int64_t* trace;                              // [4]: fwd batch, bwd batch, bwd weight version, fwd weight version
};
void tags_step(const TagOps& ops, cudaStream_t st);

void fill_f32(float* p, float v, size_t n, cudaStream_t st);
void splitk_reduce_launch(const float* partial, float* out, size_t n, int splits, bool accum, cudaStream_t st);
uint64_t launches();     // kernels launched so far through this interface

// Kernel classes for launch counting and optional device timing.
enum KernelClass {
    KC_FMA_FWD, KC_FMA_DGRAD, KC_FMA_WGRAD, KC_SPLITK, KC_BIAS_GRAD, KC_RELU_FWD, KC_RELU_BWD, KC_ADD_FWD, KC_COPY_ACC,
    KC_POOL_FWD, KC_POOL_BWD, KC_GAP_FWD, KC_GAP_BWD, KC_BN_FWD_STATS, KC_BN_FWD_APPLY, KC_BN_BWD_REDUCE, KC_BN_BWD_APPLY,
    KC_SOFTMAX_CE, KC_SGD, KC_TAGS, KC_FILL, KC_TC_FWD, KC_TC_DGRAD, KC_TC_WGRAD, KC_TC_AUX, KC_COUNT
};
struct KernelStat { uint64_t launches; double ms, flops, bytes; };
// Opened around every launch: counts it and, while profiling is enabled, records an event before and
// after it on the launching stream.  flops / bytes are the launch's ALGORITHMIC work.
struct Scope {
    int cls; cudaStream_t st; cudaEvent_t a; const char* detail;
    Scope(int cls, double flops, double bytes, cudaStream_t s);
    ~Scope();
};
void profile_detail(const char* detail);                    // tag (e.g. a layer shape) for the Scopes this thread opens next; nullptr clears
int  profile_read_detail(KernelStat* out, char (*names)[48], int capacity);   // call after profile_read
void profile_enable(bool on);                               // on: clears the statistics
int  profile_read(KernelStat* out, const char** names);     // synchronises the device; returns KC_COUNT

}  // namespace fdg
