// Step executor behind the C ABI of include/fdg.h: compiles the layer list into per-module op
// programs, lays the staleness FIFOs out in device memory, and enqueues one iteration of
// Algorithm 1 on one CUDA stream per module.
//
// FIFO layout per module k (0-based kk = k-1), D = 2(K-k)+1 (a batch forwarded at iteration
// tau+k-1 is back-propagated at iteration tau+2K-k-1, Sec. 3.2):
//   in_ring  : D+2 slots of the module's input activation.  Module k-1 writes its boundary output
//              straight into slot (tau mod (D+2)); module k reads it one iteration later for its
//              forward pass and 2(K-k) iterations after that for its backward pass.  The two extra
//              slots keep the producer's next write away from both readers without ordering the
//              forward and backward passes of an iteration.
//   stash    : D slots holding every intermediate activation (and batch-norm statistics) of the module.
//   wring    : D slots of weight versions (storage-dtype copies of the matrices + fp32 copies of the
//              vectors); version v lives in slot v mod D.
//   d2       : 2 slots of the error gradient w.r.t. the module's input; written in iteration t to
//              slot t&1, read by module k-1 in iteration t+1.
// Streams: every module has a forward stream and a backward/update stream.  Iteration t+1 of module k waits only
// for events of iteration t: its forward pass for its own update (weights, stash and ring slots it overwrites) and
// for module k-1's forward pass (its input); its backward pass for the updates of modules k+1 (error gradient) and
// k-1 (reader of the hand-off slot it overwrites); its update for its own forward pass.
#include "../../include/fdg.h"
#include "kernels.h"
#include "tc_gemm.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

using namespace fdg;

namespace {

thread_local std::string g_create_error;

enum OpType { OP_CONV, OP_BN, OP_RELU, OP_POOL, OP_GAP, OP_ADD };
enum Loc { LOC_IN, LOC_STASH, LOC_NEXT, LOC_LOGITS };

struct TensorDesc {
    int h, w, c;
    Loc loc;
    size_t off;        // byte offset inside a stash slot (LOC_STASH)
    size_t goff;       // byte offset of its gradient inside the module's gradient pool
    bool own_grad;     // gradient lives in the pool (false: d2 slot / dlogits / none)
    size_t elems() const { return (size_t)h * w * c; }
};

struct Op {
    OpType type;
    int in, in2, out;
    ConvGeom g;                    // OP_CONV
    bool bias, relu, has_res;
    size_t w_off, b_off;           // element offsets: w_off in the big segment, b_off/gamma/beta in the small segment
    size_t gamma_off, beta_off;
    size_t stats_off;              // byte offset of saved (mean, invstd) inside the stash slot (OP_BN)
    bool acc_in, acc_in2;          // backward accumulates into an already written gradient
    bool need_dgrad;
    // tensor-core plan (bf16 storage, channel counts that are multiples of 64, power-of-two images)
    bool tc;
    bool stem;                                               // thin first-layer conv: dedicated FMA kernels
    bool head;                                               // the network's last linear layer: fused with the loss (head_* kernels)
    char shape[40];                                          // "HxW Cin->Cout kR sS", the profiler's detail tag
    int n_tile_f, n_tile_d, n_tile_w, wg_splits;
    tc::KmParams kf;
    tc::KmParams kd;                                         // all output-parity classes of the input gradient in one launch
    bool dgrad_needs_zero;                                   // some parity classes receive no gradient (1x1 stride 2)
    int stat_chunks;                                         // > 0: the forward epilogue also leaves batch-norm partial sums
                                                             //      (this many per worker) for the batch-norm that follows
    tc::WgParams kw;
    std::vector<char*> a_ptrs, dy_ptrs;                      // the buffers the A / dY maps below were built for
    std::vector<char*> y_ptrs, dx_ptrs;                      // where the forward output / the input gradient can be written
    std::vector<tc::TensorMap> fo, dox;                      // output maps of the forward / input-gradient kernel, per buffer
    bool stem_tc;                                            // first layer: weight gradient on the tensor cores
    std::vector<tc::TensorMap> sxr, sdy;                     // its raw-row map of x per input buffer, its dy map
    int wgr_variant, wgr_splits;                             // rows-mode weight gradient: kernel variant (0: not used) and splits
    std::vector<tc::TensorMap> wxr;                          // x with a rows-mode box of 128-pixel steps (weight gradient)
    tc::WgRowsParams kwr;
    std::vector<tc::TensorMap> far, dar;                     // rows-mode activation maps (3x3, stride 1, tiles of whole image rows); empty: not used
    std::vector<tc::TensorMap> fa, fb, da, db, wx, wdy;      // fwd A, fwd B (per weight slot), dgrad A, dgrad B, wgrad X, wgrad dY
    std::vector<tc::TensorMap> fbh, dbh;                     // fwd / dgrad B with half-height boxes (CTA-pair kernels); empty: not used
};

struct Segment { size_t canon, internal, count; bool big; };

struct Module {
    int p, q, D, in_depth;
    int groups;                    // worker groups the op list is run for, one after the other (1 = all workers at once)
    std::vector<TensorDesc> t;
    std::vector<Op> ops;
    std::vector<Segment> segs;
    size_t n_big, n_small;         // padded element counts of the two parameter segments
    size_t in_elems;               // per-sample elements of the input / output tensor
    size_t stash_slot_bytes, wslot_bytes, grad_pool_bytes, in_slot_bytes;
    size_t ws_elems, scratch_elems, red_elems;
    char *in_ring, *stash, *gradpool, *d2, *wring, *wtring;
    float *master, *grad, *ws, *scratch, *red, *cstat;
    bool fused_update;             // one kernel per step updates all parameters and emits the next weight version (both layouts)
    tc::UpdTable upd;
    size_t cstat_elems;
    int fused_stats_tensor, fused_stats_chunks;   // set by a conv that produced statistics partials for this tensor
    int64_t *tag_in, *tag_stash, *tag_d2, *tag_w, *trace;
    cudaStream_t stream;           // backward pass, loss, update (and everything in serial mode)
    cudaStream_t fstream;          // forward pass: independent of the backward pass of the same iteration (other batch)
    cudaStream_t wstream;          // weight gradients: off the chain input gradient -> batch-norm backward -> input gradient
    cudaEvent_t wev, wdone;        // dy ready for the weight-gradient stream / its work of this iteration finished
    cudaEvent_t done, fdone, ev0, ev1;
    float* scratch_f;              // reduction scratch of the forward stream
    float* fwd_ws;                 // forward stream: partial sums of a forward pass that is split over its contraction
    size_t fwd_ws_elems;
    float* head_scratch;           // classifier head: weight-gradient partials, then loss partials
    size_t head_elems, head_part_elems;
    bool had_bwd;
};

}  // namespace

struct fdg_ctx {
    int K, n_workers, B, M, dt, esz, classes, serial, kernel_path;
    int grid_sms;                  // SMs the persistent kernels of this context size their grids for (see fdg_options.grid_sms)
    int R;                         // weight replicas per module: 1 (exact averaging, P = 11^T/N), or n_workers (general mixing matrix)
    std::vector<double> P;         // R x R mixing matrix (row-major) when R > 1
    float* P_dev;
    int in_h, in_w, in_c;
    float lr;
    int64_t t;
    bool have_params;
    bool broken;                   // a step failed after part of its work was enqueued: the FIFOs are inconsistent until fdg_set_params
    std::vector<fdg_layer> layers;
    std::vector<Module> mod;
    std::vector<void*> blocks;
    fdg_allocator alloc;
    bool own_streams;
    std::vector<cudaStream_t> owned;
    size_t n_params, device_bytes;
    int label_depth;
    int32_t* labels;
    float* logits;
    char* dlogits;
    float* loss_ring;
    int64_t* tags;
    int* tc_err;                   // device word: set by a tensor-core kernel whose bounded wait gave up
    bool any_tc;
    cudaEvent_t ingested;
    cudaEvent_t loss_ready;        // recorded behind the kernel that writes the step's loss
    std::string err;
};

namespace {

fdg_status fail(fdg_ctx* c, fdg_status s, const char* fmt, ...) {
    char buf[512];
    va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof buf, fmt, ap); va_end(ap);
    if (c) c->err = buf; else g_create_error = buf;
    return s;
}
#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(ctx, FDG_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

void* default_alloc(size_t bytes, void*) { void* p = nullptr; return cudaMalloc(&p, bytes) == cudaSuccess ? p : nullptr; }
void default_free(void* p, void*) { cudaFree(p); }

// ---- compile layers [p,q) into ops; returns "" or an error text
std::string compile_module(fdg_ctx* ctx, Module& m, int& h, int& w, int& c, bool last, size_t& canon_off) {
    const auto& L = ctx->layers;
    auto add_tensor = [&](int th, int tw, int tc) { TensorDesc d{}; d.h = th; d.w = tw; d.c = tc; d.loc = LOC_STASH; d.own_grad = true; m.t.push_back(d); return (int)m.t.size() - 1; };
    int cur = add_tensor(h, w, c);
    m.t[0].loc = LOC_IN;
    m.in_elems = m.t[0].elems();
    std::vector<int> stack;
    size_t big = 0, small = 0;
    auto seg = [&](size_t count, bool is_big) {
        size_t& pos = is_big ? big : small;
        m.segs.push_back({canon_off, pos, count, is_big});
        size_t at = pos; canon_off += count; pos += is_big ? align_up(count, 8) : align_up(count, 4);
        return at;
    };
    auto emit_conv = [&](int in, int kind, int cin, int cout, int stride, bool bias, bool relu) -> std::string {
        const TensorDesc& ti = m.t[in];
        Op o{}; o.type = OP_CONV; o.in = in; o.in2 = -1; o.bias = bias; o.relu = relu;
        ConvGeom g{};
        g.N = ctx->M;
        if (kind == FDG_LINEAR) {
            if ((size_t)cin != ti.elems()) return "linear c_in does not match the flattened input";
            g.H = g.W = 1; g.C = cin; g.R = 1; g.stride = 1; g.pad = 0;
        } else {
            if (cin != ti.c) return "conv c_in does not match the input channels";
            if (stride != 1 && stride != 2) return "stride must be 1 or 2";
            if (stride == 2 && ((ti.h | ti.w) & 1)) return "stride-2 conv needs even height and width";
            g.H = ti.h; g.W = ti.w; g.C = cin; g.R = kind == FDG_CONV3X3 ? 3 : 1; g.stride = stride; g.pad = kind == FDG_CONV3X3 ? 1 : 0;
        }
        g.Co = cout; g.Ho = (g.H + 2 * g.pad - g.R) / g.stride + 1; g.Wo = (g.W + 2 * g.pad - g.R) / g.stride + 1;
        o.g = g;
        o.w_off = seg((size_t)g.R * g.R * g.C * g.Co, true);
        if (bias) o.b_off = seg(cout, false);
        o.out = add_tensor(g.Ho, g.Wo, cout);
        std::snprintf(o.shape, sizeof o.shape, "%dx%d %d->%d k%d s%d", g.H, g.W, g.C, g.Co, g.R, g.stride);
        o.stem = ctx->kernel_path != 1 && kind == FDG_CONV3X3 && stem_supported(ctx->dt, g);
        o.stem_tc = o.stem && tc::stem_wg_supported(g.H, g.W, g.C, g.Co) && tc::init();
        // tensor-core eligibility
        int wt, ht, nt;
        o.tc = ctx->dt == 1 && ctx->kernel_path != 1 && g.C % 64 == 0 && g.Co % 64 == 0 &&
               tc::pixel_tile(g.Ho, g.Wo, 128, &wt, &ht, &nt) && g.Ho % ht == 0 && 2 * wt <= 256 && tc::init();
        if (o.tc) {
            o.n_tile_f = g.Co % 256 == 0 ? 256 : (g.Co % 128 == 0 ? 128 : 64);
            o.n_tile_d = g.C % 256 == 0 ? 256 : (g.C % 128 == 0 ? 128 : 64);
            o.n_tile_w = g.Co % 256 == 0 ? 256 : (g.Co % 128 == 0 ? 128 : 64);
            tc::pixel_tile(g.Ho, g.Wo, 64, &wt, &ht, &nt);
            int row_blocks = g.R * g.R * g.C / 64;
            long ptiles = (long)(g.Wo / wt) * (g.Ho / ht) * ((g.N + nt - 1) / nt);
            int tiles = ((row_blocks + 1) / 2) * (g.Co / o.n_tile_w);
            long want = ((o.n_tile_w == 64 ? 4 : 2) * ctx->grid_sms) / tiles;   // CTAs = tiles * splits fill whole waves of the context's SMs (two CTAs per SM fit for the 64-column tile)
            long splits = want < 1 ? 1 : want;
            if (splits > ptiles) splits = ptiles;
            long pps = (ptiles + splits - 1) / splits;
            o.wg_splits = (int)((ptiles + pps - 1) / pps);
            o.wgr_variant = (g.R == 3 && g.stride == 1) ? tc::wg_rows_variant(g.H, g.W, g.C, g.Co) : 0;
            if (o.wgr_variant) {
                tc::pixel_tile(g.Ho, g.Wo, 128, &wt, &ht, &nt);
                o.wgr_splits = tc::wg_rows_splits(o.wgr_variant, g.C, g.Co, (long)(g.Ho / ht) * ((g.N + nt - 1) / nt), ctx->grid_sms);
            }
        }
        m.ops.push_back(o);
        return "";
    };
    auto emit_bn = [&](int in, int in2, bool relu) {
        Op o{}; o.type = OP_BN; o.in = in; o.in2 = in2; o.has_res = in2 >= 0; o.relu = relu;
        const TensorDesc ti = m.t[in];
        o.g = ConvGeom{}; o.g.C = ti.c;
        o.gamma_off = seg(ti.c, false); o.beta_off = seg(ti.c, false);
        o.out = add_tensor(ti.h, ti.w, ti.c);
        m.ops.push_back(o);
        return o.out;
    };
    // a projecting shortcut: conv1x1(stride) + batch-norm of the saved block input
    auto emit_shortcut = [&](const fdg_layer& Y, int sc, std::string& err) -> int {
        if (!(Y.flags & 1)) return sc;
        err = emit_conv(sc, FDG_CONV1X1, Y.c_in, Y.c_out, Y.stride, false, false);
        if (!err.empty()) return -1;
        return emit_bn(m.ops.back().out, -1, false);
    };

    for (int l = m.p; l < m.q; ++l) {
        const fdg_layer& Y = L[l];
        const TensorDesc tc = m.t[cur];
        auto next_is = [&](int kind) { return l + 1 < m.q && L[l + 1].kind == kind; };
        switch (Y.kind) {
            case FDG_LINEAR: case FDG_CONV3X3: case FDG_CONV1X1: {
                bool relu = next_is(FDG_RELU);
                std::string e = emit_conv(cur, Y.kind, Y.c_in, Y.c_out, Y.stride, Y.flags & 1, relu);
                if (!e.empty()) return e;
                cur = m.ops.back().out;
                if (relu) ++l;
                break; }
            case FDG_BATCHNORM: {
                if (Y.c_in != tc.c) return "batch-norm channel count does not match";
                if (next_is(FDG_RES_ADD)) {
                    // canonical order: the batch-norm's gamma/beta come before the shortcut's parameters
                    const fdg_layer& A = L[l + 1];
                    if (stack.empty()) return "RES_ADD without RES_BEGIN";
                    int sc = stack.back(); stack.pop_back();
                    size_t gcan = canon_off; canon_off += 2 * (size_t)tc.c;         // reserve gamma, beta
                    std::string e; int s2 = emit_shortcut(A, sc, e);
                    if (!e.empty()) return e;
                    const TensorDesc ts = m.t[s2];
                    if (ts.h != tc.h || ts.w != tc.w || ts.c != tc.c) return "shortcut shape does not match the block output";
                    l += 1;
                    bool relu = next_is(FDG_RELU);
                    size_t after = canon_off; canon_off = gcan;
                    cur = emit_bn(cur, s2, relu);
                    canon_off = after;
                    if (relu) ++l;
                } else {
                    bool relu = next_is(FDG_RELU);
                    cur = emit_bn(cur, -1, relu);
                    if (relu) ++l;
                }
                break; }
            case FDG_RELU: { Op o{}; o.type = OP_RELU; o.in = cur; o.in2 = -1; o.out = add_tensor(tc.h, tc.w, tc.c); m.ops.push_back(o); cur = o.out; break; }
            case FDG_MAXPOOL2: {
                if ((tc.h | tc.w) & 1) return "max-pool needs even height and width";
                Op o{}; o.type = OP_POOL; o.in = cur; o.in2 = -1; o.out = add_tensor(tc.h / 2, tc.w / 2, tc.c); m.ops.push_back(o); cur = o.out; break; }
            case FDG_GLOBAL_AVGPOOL: { Op o{}; o.type = OP_GAP; o.in = cur; o.in2 = -1; o.out = add_tensor(1, 1, tc.c); m.ops.push_back(o); cur = o.out; break; }
            case FDG_RES_BEGIN: stack.push_back(cur); break;
            case FDG_RES_ADD: {
                if (stack.empty()) return "RES_ADD without RES_BEGIN";
                int sc = stack.back(); stack.pop_back();
                std::string e; int s2 = emit_shortcut(Y, sc, e);
                if (!e.empty()) return e;
                const TensorDesc ts = m.t[s2];
                if (ts.h != tc.h || ts.w != tc.w || ts.c != tc.c) return "shortcut shape does not match the block output";
                Op o{}; o.type = OP_ADD; o.in = cur; o.in2 = s2; o.out = add_tensor(tc.h, tc.w, tc.c); m.ops.push_back(o); cur = o.out; break; }
            default: return "unknown layer kind";
        }
    }
    if (!stack.empty()) return "BAD_SPLIT: a split point cuts a residual block";
    if (m.ops.empty()) return "a module has no computing layer";
    if (m.ops.back().out != cur) return "internal: dangling tensor";
    h = m.t[cur].h; w = m.t[cur].w; c = m.t[cur].c;
    m.head_elems = m.head_part_elems = 0;
    if (last) {
        Op& o = m.ops.back();
        if (o.type != OP_CONV || o.relu || o.g.Ho * o.g.Wo != 1) return "the network must end with a linear layer";
        m.t[cur].loc = LOC_LOGITS;
        if (o.g.H * o.g.W == 1 && o.g.R == 1 && head_supported(ctx->dt, o.g.C, o.g.Co)) {
            o.head = true; o.tc = false; o.stem = false; o.stem_tc = false;
            m.head_elems = head_scratch_elems(ctx->M, o.g.C, o.g.Co);
            m.head_part_elems = m.head_elems - (size_t)(ctx->M + 7) / 8;
        }
    } else {
        m.t[cur].loc = LOC_NEXT;
    }
    m.t[cur].own_grad = false;
    m.t[0].own_grad = false;
    m.n_big = big; m.n_small = small;

    // stash layout, gradient pool layout, scratch sizes
    size_t soff = 0, goff = 0;
    for (size_t i = 0; i < m.t.size(); ++i) {
        TensorDesc& d = m.t[i];
        if (d.loc == LOC_STASH) { d.off = soff; soff += align_up(d.elems() * ctx->M * ctx->esz, 256); }
        if (d.own_grad) { d.goff = goff; goff += align_up(d.elems() * ctx->M * ctx->esz, 256); }
    }
    m.ws_elems = 0; m.scratch_elems = 64; m.red_elems = 4; m.fwd_ws_elems = 0;
    for (Op& o : m.ops) {
        if (o.type == OP_BN) {
            o.stats_off = soff; soff += align_up((size_t)ctx->n_workers * o.g.C * 2 * sizeof(float), 256);
            m.scratch_elems = std::max(m.scratch_elems, (size_t)128 * ctx->n_workers * o.g.C * 2);
            m.red_elems = std::max(m.red_elems, (size_t)ctx->n_workers * o.g.C * 2);
        }
        if (o.type == OP_CONV) {
            if (o.tc) m.ws_elems = std::max(m.ws_elems, (size_t)std::max(o.wg_splits, o.wgr_variant ? o.wgr_splits : 0) * o.g.R * o.g.R * o.g.C * o.g.Co);
            if (o.stem) m.ws_elems = std::max(m.ws_elems, stem_wgrad_workspace_elems(o.g));
            if (o.stem_tc) m.ws_elems = std::max(m.ws_elems, tc::stem_wg_workspace_elems(o.g.Co, (long)o.g.N * o.g.H, ctx->grid_sms));
            m.ws_elems = std::max(m.ws_elems, wgrad_workspace_elems(o.g));
            m.fwd_ws_elems = std::max(m.fwd_ws_elems, forward_workspace_elems(o.g));
            m.scratch_elems = std::max(m.scratch_elems, (size_t)64 * o.g.Co);
            if (relu_bias_backward_supported(ctx->dt, o.g.Co)) m.scratch_elems = std::max(m.scratch_elems, relu_bias_backward_scratch_elems(o.g.Co));
        }
    }
    // a tensor-core conv whose output goes straight into a batch-norm computes that batch-norm's statistics
    // in its epilogue, if its 128-row tiles never straddle two workers
    m.cstat_elems = 0;
    for (size_t i = 0; i + 1 < m.ops.size(); ++i) {
        Op& o = m.ops[i];
        const Op& nx = m.ops[i + 1];
        o.stat_chunks = 0;
        if (o.type != OP_CONV || !(o.tc || o.stem_tc) || nx.type != OP_BN || nx.in != o.out || !bn_accepts_conv_partials(ctx->dt, o.g.Co)) continue;
        int wt, ht, nt;
        tc::pixel_tile(o.g.Ho, o.g.Wo, 128, &wt, &ht, &nt);
        if (ctx->B % nt != 0) continue;
        o.stat_chunks = (ctx->B / nt) * (o.g.Ho / ht) * (o.g.Wo / wt) * 4;
        m.cstat_elems = std::max(m.cstat_elems, (size_t)ctx->n_workers * o.stat_chunks * o.g.Co * 2);
    }
    m.stash_slot_bytes = align_up(soff, 256);
    m.grad_pool_bytes = align_up(goff, 256);
    // backward write/accumulate analysis: walking the ops in reverse, the first op that touches a
    // tensor's gradient writes it, later ones add to it
    std::vector<char> written(m.t.size(), 0);
    for (int i = (int)m.ops.size() - 1; i >= 0; --i) {
        Op& o = m.ops[i];
        o.acc_in = written[o.in]; written[o.in] = 1;
        if (o.in2 >= 0) { o.acc_in2 = written[o.in2]; written[o.in2] = 1; }
        o.need_dgrad = true;
    }
    return "";
}

struct StepPtrs {            // resolved addresses for one (module, batch)
    fdg_ctx* c; Module* m; int kk;
    int64_t batch;
    char* tensor(int id) const {
        const TensorDesc& d = m->t[id];
        switch (d.loc) {
            case LOC_IN: return m->in_ring + (size_t)(batch % m->in_depth) * m->in_slot_bytes;
            case LOC_STASH: return m->stash + (size_t)(batch % m->D) * m->stash_slot_bytes + d.off;
            case LOC_NEXT: { Module& n = c->mod[kk + 1]; return n.in_ring + (size_t)(batch % n.in_depth) * n.in_slot_bytes; }
            case LOC_LOGITS: return (char*)c->logits;
        }
        return nullptr;
    }
    float* stats(const Op& o) const { return (float*)(m->stash + (size_t)(batch % m->D) * m->stash_slot_bytes + o.stats_off); }
};

// weight version `version` of replica r (r = 0 unless the context keeps one replica per worker)
char* wslot(fdg_ctx* c, Module& m, int64_t version, int r = 0) { return m.wring + ((size_t)(version % m.D) * c->R + r) * m.wslot_bytes; }
char* wbig(fdg_ctx* c, Module& m, int64_t version, size_t off, int r = 0) { return wslot(c, m, version, r) + off * c->esz; }
float* wsmall(fdg_ctx* c, Module& m, int64_t version, size_t off, int r = 0) { return (float*)(wslot(c, m, version, r) + m.n_big * c->esz) + off; }
size_t npar(const Module& m) { return m.n_big + m.n_small; }

char* wtslot(Module& m, int64_t version, size_t off) { return m.wtring + ((size_t)(version % m.D) * m.n_big + off) * 2; }

int find_buf(const std::vector<char*>& v, const char* p) {
    for (size_t i = 0; i < v.size(); ++i) if (v[i] == p) return (int)i;
    return -1;
}

// forward conv / linear on the tensor cores; false if the buffers are not the ones planned for
// A group of consecutive workers (rows n0 .. n0+n-1 of every [M, ...] tensor).  A module whose tensors are far
// larger than L2 runs its op list once per group, so that what one kernel writes is still in L2 when the next
// kernel reads it; weight / bias / gamma / beta gradients of the second and later groups add to the first's.
struct Win { int n0, n, w0, nw; bool first; };

Win group_window(const fdg_ctx* c, const Module& m, int g) {
    const int nw = c->n_workers / m.groups;
    return Win{g * nw * c->B, nw * c->B, g * nw, nw, g == 0};
}

bool tc_forward(fdg_ctx* c, Module& m, const Op& o, char* x_base, char* y_base, int64_t version, const Win& wn, cudaStream_t s) {
    int ia = find_buf(o.a_ptrs, x_base);
    if (ia < 0) return false;
    tc::KmParams p = o.kf;
    p.bias = o.bias ? wsmall(c, m, version, o.b_off) : nullptr;
    p.out = y_base; p.epi = o.relu ? EPI_RELU : 0; p.err = c->tc_err; p.sms = c->grid_sms;
    p.stat_part = o.stat_chunks ? m.cstat : nullptr;
    p.n_base = wn.n0; p.N = wn.n0 + wn.n; p.tiles_n = (wn.n + p.Nt - 1) / p.Nt;
    const ConvGeom& g = o.g;
    double rows = (double)wn.n * g.Ho * g.Wo;
    Scope sc(KC_TC_FWD, 2.0 * rows * g.Co * g.R * g.R * g.C, 2.0 * ((double)wn.n * g.H * g.W * g.C + (double)g.Co * g.R * g.R * g.C + rows * g.Co), s);
    const int io = find_buf(o.y_ptrs, y_base);
    const tc::KmMaps maps{&o.fa[ia], o.far.empty() ? nullptr : &o.far[ia], &o.fb[version % m.D], o.fbh.empty() ? nullptr : &o.fbh[version % m.D],
                          io >= 0 ? &o.fo[io] : nullptr};
    const bool ok = tc::run_km(maps, p, o.n_tile_f, s) == cudaSuccess;
    if (ok && o.stat_chunks) { m.fused_stats_tensor = o.out; m.fused_stats_chunks = o.stat_chunks; }
    return ok;
}
bool tc_dgrad(fdg_ctx* c, Module& m, const Op& o, char* dy_base, char* dx_base, int64_t version, bool accum, const Win& wn, cudaStream_t s) {
    int ia = find_buf(o.dy_ptrs, dy_base);
    if (ia < 0) return false;
    const ConvGeom& g = o.g;
    double rows = (double)wn.n * g.H * g.W;
    if (o.dgrad_needs_zero && !accum) {
        Scope sc(KC_TC_AUX, 0.0, 2.0 * rows * g.C, s);
        cudaMemsetAsync(dx_base + (size_t)wn.n0 * g.H * g.W * g.C * 2, 0, (size_t)rows * g.C * 2, s);
    }
    tc::KmParams p = o.kd;
    p.bias = nullptr; p.out = dx_base; p.epi = accum ? EPI_ACCUM : 0; p.err = c->tc_err; p.stat_part = nullptr; p.sms = c->grid_sms;
    p.n_base = wn.n0; p.N = wn.n0 + wn.n; p.tiles_n = (wn.n + p.Nt - 1) / p.Nt;
    const double crows = (double)wn.n * p.Hd * p.Wd;         // pixels of one class; every tap belongs to exactly one class
    Scope sc(KC_TC_DGRAD, 2.0 * crows * g.C * p.ntaps * g.Co,
             2.0 * ((double)wn.n * g.Ho * g.Wo * g.Co + (double)g.Co * p.ntaps * g.C + crows * p.ncls * g.C * (accum ? 2 : 1)), s);
    const int io = find_buf(o.dx_ptrs, dx_base);
    const tc::KmMaps maps{&o.da[ia], o.dar.empty() ? nullptr : &o.dar[ia], &o.db[version % m.D], o.dbh.empty() ? nullptr : &o.dbh[version % m.D],
                          io >= 0 ? &o.dox[io] : nullptr};
    return tc::run_km(maps, p, o.n_tile_d, s) == cudaSuccess;
}
bool tc_wgrad(fdg_ctx* c, Module& m, const Op& o, char* x_base, char* dy_base, float* dw, const Win& wn, cudaStream_t s) {
    int ix = find_buf(o.a_ptrs, x_base), id = find_buf(o.dy_ptrs, dy_base);
    if (ix < 0 || id < 0) return false;
    const ConvGeom& g = o.g;
    if (o.wgr_variant && wn.n % o.kwr.Nt == 0) {
        tc::WgRowsParams q = o.kwr;
        q.partial = m.ws; q.err = c->tc_err; q.n_base = wn.n0; q.tiles_n = wn.n / q.Nt;
        const long steps = (long)q.tiles_h * q.tiles_n;
        const int splits = o.wgr_splits < steps ? o.wgr_splits : (int)steps;
        double rows = (double)wn.n * g.Ho * g.Wo, R = (double)g.R * g.R * g.C;
        Scope sc(KC_TC_WGRAD, 2.0 * rows * g.Co * R, 2.0 * ((double)wn.n * g.H * g.W * g.C + rows * g.Co) + 4.0 * R * g.Co, s);
        return tc::run_wg_rows(o.wxr[ix], o.da[id], q, o.wgr_variant, splits, dw, !wn.first, s) == cudaSuccess;
    }
    tc::WgParams p = o.kw;
    p.partial = m.ws; p.err = c->tc_err;
    p.n_base = wn.n0; p.tiles_n = (wn.n + p.Nt - 1) / p.Nt;
    p.ptiles = p.tiles_w * p.tiles_h * p.tiles_n;
    int splits = o.wg_splits < p.ptiles ? o.wg_splits : p.ptiles;
    p.ptiles_per_split = (p.ptiles + splits - 1) / splits;
    splits = (p.ptiles + p.ptiles_per_split - 1) / p.ptiles_per_split;
    double rows = (double)wn.n * g.Ho * g.Wo, R = (double)g.R * g.R * g.C;
    Scope sc(KC_TC_WGRAD, 2.0 * rows * g.Co * R, 2.0 * ((double)wn.n * g.H * g.W * g.C + rows * g.Co) + 4.0 * R * g.Co, s);
    return tc::run_wg(o.wx[ix], o.wdy[id], p, o.n_tile_w, splits, dw, !wn.first, s) == cudaSuccess;
}

// first-layer forward on the tensor cores (whole batch only)
bool tc_stem_forward(fdg_ctx* c, Module& m, const Op& o, char* x_base, char* y_base, int64_t version, const Win& wn, cudaStream_t s) {
    if (!o.stem_tc || wn.n != c->M) return false;
    const int ix = find_buf(o.a_ptrs, x_base), io = find_buf(o.y_ptrs, y_base);
    if (ix < 0 || io < 0) return false;
    const ConvGeom& g = o.g;
    const double pix = (double)g.N * g.H * g.W;
    Scope sc(KC_FMA_FWD, 2.0 * pix * g.Co * 9 * g.C, 2.0 * pix * (g.C + g.Co), s);
    const bool ok = tc::run_stem_fw(o.sxr[ix], o.fo[io], g.H, g.W, g.N, g.Co, wbig(c, m, version, o.w_off), o.bias ? wsmall(c, m, version, o.b_off) : nullptr,
                                    o.relu, o.stat_chunks ? m.cstat : nullptr, c->tc_err, c->grid_sms, s) == cudaSuccess;
    if (ok && o.stat_chunks) { m.fused_stats_tensor = o.out; m.fused_stats_chunks = o.stat_chunks; }
    return ok;
}

// first-layer weight gradient on the tensor cores (whole batch only)
bool tc_stem_wgrad(fdg_ctx* c, Module& m, const Op& o, char* x_base, char* dy_base, float* dw, const Win& wn, cudaStream_t s) {
    if (!o.stem_tc || wn.n != c->M) return false;
    const int ix = find_buf(o.a_ptrs, x_base), id = find_buf(o.dy_ptrs, dy_base);
    if (ix < 0 || id < 0) return false;
    const ConvGeom& g = o.g;
    const double pix = (double)g.N * g.H * g.W;
    Scope sc(KC_FMA_WGRAD, 2.0 * pix * g.Co * 9 * g.C, 2.0 * pix * (g.C + g.Co), s);
    return tc::run_stem_wg(o.sxr[ix], o.sdy[id], g.H, g.W, g.N, g.Co, m.ws, dw, false, c->tc_err, c->grid_sms, s) == cudaSuccess;
}

// byte offset of the group's first sample inside a tensor of the module
size_t row_off(const fdg_ctx* c, const TensorDesc& d, const Win& wn) {
    return (size_t)wn.n0 * d.elems() * (d.loc == LOC_LOGITS ? sizeof(float) : (size_t)c->esz);
}

void forward_module(fdg_ctx* c, int kk, int64_t batch, int64_t version, int group) {
    Module& m = c->mod[kk];
    StepPtrs P{c, &m, kk, batch};
    const Win wn = group_window(c, m, group);
    const int rep = c->R > 1 ? group : 0;               // worker `group` runs on its own weights w_{s,k}
    cudaStream_t s = m.fstream;
    const int dt = c->dt;
    m.fused_stats_tensor = -1;
    auto T = [&](int id) { return P.tensor(id) + row_off(c, m.t[id], wn); };
    for (const Op& o : m.ops) {
        const TensorDesc& ti = m.t[o.in];
        const TensorDesc& to = m.t[o.out];
        size_t n_out = to.elems() * wn.n;
        switch (o.type) {
            case OP_CONV: {
                int epi = (o.relu ? EPI_RELU : 0) | (to.loc == LOC_LOGITS ? EPI_OUT_F32 : 0);
                ConvGeom g = o.g; g.N = wn.n;
                profile_detail(o.shape);
                if (o.head && m.groups == 1) {
                    // logits, loss and dphi/dlogits / M of batch `batch` in one launch (version == the iteration t)
                    head_forward_loss(dt, T(o.in), wbig(c, m, version, o.w_off), o.bias ? wsmall(c, m, version, o.b_off) : nullptr,
                                      c->labels + (size_t)(batch % c->label_depth) * c->M, c->logits, c->dlogits, m.head_scratch + m.head_part_elems,
                                      (unsigned*)(c->tc_err + 16), c->loss_ring + (version % 64), c->M, g.C, g.Co, 1.f / (float)c->M, s);
                    profile_detail(nullptr);
                    break;
                }
                if (o.tc && tc_forward(c, m, o, P.tensor(o.in), P.tensor(o.out), version, wn, s)) { profile_detail(nullptr); break; }
                if (o.stem && tc_stem_forward(c, m, o, P.tensor(o.in), P.tensor(o.out), version, wn, s)) { profile_detail(nullptr); break; }
                if (o.stem) {
                    stem_forward(T(o.in), wbig(c, m, version, o.w_off, rep), o.bias ? wsmall(c, m, version, o.b_off, rep) : nullptr, T(o.out), g, o.relu, s);
                    profile_detail(nullptr);
                    break;
                }
                conv_forward(dt, T(o.in), wbig(c, m, version, o.w_off, rep), o.bias ? wsmall(c, m, version, o.b_off, rep) : nullptr, T(o.out), g, epi,
                             m.fwd_ws, m.fwd_ws_elems, s);
                profile_detail(nullptr);
                break; }
            case OP_BN: {
                char tag[40];
                std::snprintf(tag, sizeof tag, "%dx%dx%d%s%s", ti.h, ti.w, ti.c, o.has_res ? " +res" : "", o.relu ? " relu" : "");
                profile_detail(tag);
                const bool fused = m.fused_stats_tensor == o.in;
                const float* part = fused ? m.cstat + (size_t)wn.w0 * m.fused_stats_chunks * ti.c * 2 : nullptr;
                bn_forward(dt, T(o.in), wsmall(c, m, version, o.gamma_off, rep), wsmall(c, m, version, o.beta_off, rep),
                           o.has_res ? T(o.in2) : nullptr, T(o.out), P.stats(o) + (size_t)wn.w0 * ti.c * 2, m.scratch_f, wn.nw,
                           (long)c->B * ti.h * ti.w, ti.c, o.relu, part, fused ? m.fused_stats_chunks : 0, c->grid_sms, c->tc_err, s);
                profile_detail(nullptr);
                m.fused_stats_tensor = -1;
                break; }
            case OP_RELU: relu_forward(dt, T(o.in), T(o.out), n_out, s); break;
            case OP_POOL: maxpool_forward(dt, T(o.in), T(o.out), wn.n, ti.h, ti.w, ti.c, s); break;
            case OP_GAP: gap_forward(dt, T(o.in), T(o.out), wn.n, ti.h * ti.w, ti.c, s); break;
            case OP_ADD: add_forward(dt, T(o.in), T(o.in2), T(o.out), n_out, s); break;
        }
    }
}

// gradient buffer of a tensor during iteration t
char* grad_ptr(fdg_ctx* c, int kk, int id, int64_t t) {
    Module& m = c->mod[kk];
    const TensorDesc& d = m.t[id];
    if (d.own_grad) return m.gradpool + d.goff;
    if (id == 0) return kk > 0 ? m.d2 + (size_t)(t & 1) * m.in_slot_bytes : nullptr;          // sent to module k-1
    if (d.loc == LOC_LOGITS) return c->dlogits;
    Module& n = c->mod[kk + 1];                                                                // received from module k+1
    return n.d2 + (size_t)((t - 1) & 1) * n.in_slot_bytes;
}

void backward_module(fdg_ctx* c, int kk, int64_t batch, int64_t version, int64_t t, int group) {
    Module& m = c->mod[kk];
    StepPtrs P{c, &m, kk, batch};
    const Win wn = group_window(c, m, group);
    cudaStream_t s = m.stream;
    const int dt = c->dt;
    const int rep = c->R > 1 ? group : 0;
    const bool acc_p = c->R > 1 ? false : !wn.first;    // one replica: parameter gradients of later groups add to the first group's
    float* const mgrad = m.grad + (size_t)rep * npar(m); // g_{s,k} of this replica
    auto T = [&](int id) { return P.tensor(id) + row_off(c, m.t[id], wn); };
    // gradients are stored in the storage dtype (also the one of the logits)
    auto G = [&](int id) -> char* { char* b = grad_ptr(c, kk, id, t); return b ? b + (size_t)wn.n0 * m.t[id].elems() * c->esz : nullptr; };
    for (int i = (int)m.ops.size() - 1; i >= 0; --i) {
        const Op& o = m.ops[i];
        const TensorDesc& ti = m.t[o.in];
        const TensorDesc& to = m.t[o.out];
        size_t n_out = to.elems() * wn.n, n_in = ti.elems() * wn.n;
        char* gout = G(o.out);
        char* gin = G(o.in);
        switch (o.type) {
            case OP_CONV: {
                ConvGeom g = o.g; g.N = wn.n;
                if (o.head && m.groups == 1) {
                    profile_detail(o.shape);
                    head_backward(dt, T(o.in), wbig(c, m, version, o.w_off), gout, gin, o.acc_in, mgrad + o.w_off, o.bias ? mgrad + m.n_big + o.b_off : nullptr,
                                  m.head_scratch, c->M, g.C, g.Co, s);
                    profile_detail(nullptr);
                    break;
                }
                // dZ = dA * (A > 0) in place and the bias gradient, in one pass over dA where the width allows
                const long orows = (long)g.N * g.Ho * g.Wo;
                const bool fused_rb = (o.relu || o.bias) && relu_bias_backward_supported(dt, g.Co);
                if (fused_rb) relu_bias_backward(dt, o.relu ? T(o.out) : nullptr, gout, o.bias ? mgrad + m.n_big + o.b_off : nullptr, m.scratch, orows, g.Co, acc_p, s);
                else if (o.relu) relu_backward(dt, T(o.out), gout, gout, n_out, false, s);
                profile_detail(o.shape);
                // the weight gradient needs dy as it stands now and is needed only by the update: it goes to its own stream
                cudaStream_t ws = m.wstream;
                if (ws != s) { cudaEventRecord(m.wev, s); cudaStreamWaitEvent(ws, m.wev, 0); }
                if (o.stem && tc_stem_wgrad(c, m, o, P.tensor(o.in), grad_ptr(c, kk, o.out, t), mgrad + o.w_off, wn, ws)) {}
                else if (o.stem) stem_wgrad(T(o.in), gout, mgrad + o.w_off, m.ws, g, acc_p, ws);
                else if (!(o.tc && tc_wgrad(c, m, o, P.tensor(o.in), grad_ptr(c, kk, o.out, t), mgrad + o.w_off, wn, ws)))
                    conv_wgrad(dt, T(o.in), gout, mgrad + o.w_off, m.ws, g, acc_p, ws);
                if (o.bias && !fused_rb) bias_grad(dt, gout, mgrad + m.n_big + o.b_off, m.scratch, orows, g.Co, acc_p, s);
                if (gin && !(o.tc && tc_dgrad(c, m, o, grad_ptr(c, kk, o.out, t), grad_ptr(c, kk, o.in, t), version, o.acc_in, wn, s)))
                    conv_dgrad(dt, gout, wbig(c, m, version, o.w_off, rep), gin, g, o.acc_in ? EPI_ACCUM : 0, s);
                profile_detail(nullptr);
                break; }
            case OP_BN: {
                char tag[40];
                std::snprintf(tag, sizeof tag, "%dx%dx%d%s%s", ti.h, ti.w, ti.c, o.has_res ? " +res" : "", o.relu ? " relu" : "");
                profile_detail(tag);
                char* gres = o.has_res ? G(o.in2) : nullptr;
                bn_backward(dt, T(o.in), T(o.out), gout, wsmall(c, m, version, o.gamma_off, rep), wsmall(c, m, version, o.beta_off, rep),
                            P.stats(o) + (size_t)wn.w0 * ti.c * 2, gin, o.acc_in, gres, o.acc_in2, mgrad + m.n_big + o.gamma_off,
                            mgrad + m.n_big + o.beta_off, m.red, m.scratch, wn.nw, (long)c->B * ti.h * ti.w, ti.c, o.relu, o.has_res, acc_p, c->grid_sms, c->tc_err, s);
                profile_detail(nullptr);
                break; }
            case OP_RELU: if (gin) relu_backward(dt, T(o.out), gout, gin, n_out, o.acc_in, s); break;
            case OP_POOL: if (gin) maxpool_backward(dt, T(o.in), gout, gin, wn.n, ti.h, ti.w, ti.c, o.acc_in, s); break;
            case OP_GAP: if (gin) gap_backward(dt, gout, gin, wn.n, ti.h * ti.w, ti.c, o.acc_in, s); break;
            case OP_ADD: {
                if (gin) copy_or_accumulate(dt, gout, gin, n_in, o.acc_in, s);
                char* g2 = G(o.in2);
                if (g2) copy_or_accumulate(dt, gout, g2, n_in, o.acc_in2, s);
                break; }
        }
    }
}

// Emit the transposed (and tap-flipped) copies of weight version `version` that the input-gradient kernel reads.
void emit_transposed_weights(fdg_ctx* c, Module& m, int64_t version) {
    for (const Op& o : m.ops)
        if (o.type == OP_CONV && o.tc) {
            Scope sc(KC_TC_AUX, 0.0, 4.0 * o.g.R * o.g.R * o.g.C * o.g.Co, m.stream);
            tc::run_flip_transpose(wbig(c, m, version, o.w_off), wtslot(m, version, o.w_off), o.g.Co, o.g.R * o.g.R, o.g.C, m.stream);
        }
}

// Build the TMA tensor maps of every tensor-core op (needs the final device addresses).
bool build_tc_plans(fdg_ctx* c) {
    for (int kk = 0; kk < c->K; ++kk) {
        Module& m = c->mod[kk];
        for (Op& o : m.ops) {
            if (o.type == OP_CONV && o.stem_tc) {
                const ConvGeom& g = o.g;
                const TensorDesc& ti = m.t[o.in];
                const TensorDesc& to = m.t[o.out];
                if (ti.loc == LOC_IN) for (int i = 0; i < m.in_depth; ++i) o.a_ptrs.push_back(m.in_ring + (size_t)i * m.in_slot_bytes);
                else for (int i = 0; i < m.D; ++i) o.a_ptrs.push_back(m.stash + (size_t)i * m.stash_slot_bytes + ti.off);
                if (to.own_grad) o.dy_ptrs.push_back(m.gradpool + to.goff);
                else if (to.loc == LOC_NEXT) { Module& n = c->mod[kk + 1]; for (int i = 0; i < 2; ++i) o.dy_ptrs.push_back(n.d2 + (size_t)i * n.in_slot_bytes); }
                int wt, ht, nt;
                tc::pixel_tile(g.Ho, g.Wo, 128, &wt, &ht, &nt);
                bool ok = true;
                o.sxr.resize(o.a_ptrs.size()); o.sdy.resize(o.dy_ptrs.size());
                for (size_t i = 0; i < o.a_ptrs.size(); ++i) ok = ok && tc::make_map_raw_rows(&o.sxr[i], o.a_ptrs[i], g.C, g.W, g.H, g.N, ht + 2);
                for (size_t i = 0; i < o.dy_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.sdy[i], o.dy_ptrs[i], g.Co, g.Wo, g.Ho, g.N, 64, wt, ht, nt, 1);
                if (to.loc == LOC_STASH) for (int i = 0; i < m.D; ++i) o.y_ptrs.push_back(m.stash + (size_t)i * m.stash_slot_bytes + to.off);
                else if (to.loc == LOC_NEXT) { Module& n = c->mod[kk + 1]; for (int i = 0; i < n.in_depth; ++i) o.y_ptrs.push_back(n.in_ring + (size_t)i * n.in_slot_bytes); }
                o.fo.resize(o.y_ptrs.size());
                for (size_t i = 0; i < o.y_ptrs.size(); ++i) ok = ok && tc::make_map_out(&o.fo[i], o.y_ptrs[i], g.Co, g.Wo, g.Ho, g.N, wt, ht);
                if (!ok || o.dy_ptrs.empty() || o.y_ptrs.empty()) { o.stem_tc = false; o.stat_chunks = 0; continue; }
                c->any_tc = true;
                continue;
            }
            if (o.type != OP_CONV || !o.tc) continue;
            const ConvGeom& g = o.g;
            const TensorDesc& ti = m.t[o.in];
            const TensorDesc& to = m.t[o.out];
            // where the input activation can live
            if (ti.loc == LOC_IN) for (int i = 0; i < m.in_depth; ++i) o.a_ptrs.push_back(m.in_ring + (size_t)i * m.in_slot_bytes);
            else for (int i = 0; i < m.D; ++i) o.a_ptrs.push_back(m.stash + (size_t)i * m.stash_slot_bytes + ti.off);
            // where the output gradient can live
            if (to.own_grad) o.dy_ptrs.push_back(m.gradpool + to.goff);
            else if (to.loc == LOC_NEXT) { Module& n = c->mod[kk + 1]; for (int i = 0; i < 2; ++i) o.dy_ptrs.push_back(n.d2 + (size_t)i * n.in_slot_bytes); }
            else { o.tc = false; continue; }
            int wt, ht, nt;
            const int taps = g.R * g.R, Ktot = taps * g.C;
            bool ok = true;
            // ---- forward: A = x (128-pixel boxes), B = W [Co][taps*C]
            tc::pixel_tile(g.Ho, g.Wo, 128, &wt, &ht, &nt);
            tc::KmParams& f = o.kf; f = tc::KmParams{};
            f.Wt = wt; f.Ht = ht; f.Nt = nt; f.tiles_w = g.Wo / wt; f.tiles_h = g.Ho / ht; f.tiles_n = (g.N + nt - 1) / nt;
            f.ntaps = taps; f.kchunks = g.C / 64; f.xs = g.stride;
            for (int t = 0; t < taps; ++t) { f.dh[t] = t / g.R - g.pad; f.dw[t] = t % g.R - g.pad; f.koff[t] = t * g.C; }
            f.N = g.N; f.Hd = g.Ho; f.Wd = g.Wo; f.Ho = g.Ho; f.Wo = g.Wo; f.Co = g.Co; f.os = 1; f.Cn = g.Co;
            f.ncls = 1; f.cls_tap0[0] = 0; f.cls_tap0[1] = taps; f.cls_oph[0] = 0; f.cls_opw[0] = 0;
            o.fa.resize(o.a_ptrs.size());
            for (size_t i = 0; i < o.a_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.fa[i], o.a_ptrs[i], g.C, g.W, g.H, g.N, 64, wt, ht, nt, g.stride);
            // rows mode: a box of the tile's rows plus one above and one below, for a tile that is whole rows of one image
            const bool rows_ok = g.R == 3 && g.stride == 1 && wt == g.Wo && nt == 1 && (ht + 2) * g.Wo * 128 <= 24 * 1024;   // the stage holds ht + 2 rows of 128-byte pixels in 24 KB
            if (rows_ok) {
                o.far.resize(o.a_ptrs.size());
                for (size_t i = 0; i < o.a_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.far[i], o.a_ptrs[i], g.C, g.W, g.H, g.N, 64, g.W, ht + 2, 1, 1);
            }
            o.fb.resize(m.D);
            for (int v = 0; v < m.D; ++v) ok = ok && tc::make_map_2d(&o.fb[v], wbig(c, m, v, o.w_off), Ktot, g.Co, 64, o.n_tile_f);
            f.Nfull = g.N;
            // the forward output: a stash slot, or a slot of the next module's input ring
            if (to.loc == LOC_STASH) for (int i = 0; i < m.D; ++i) o.y_ptrs.push_back(m.stash + (size_t)i * m.stash_slot_bytes + to.off);
            else if (to.loc == LOC_NEXT) { Module& n = c->mod[kk + 1]; for (int i = 0; i < n.in_depth; ++i) o.y_ptrs.push_back(n.in_ring + (size_t)i * n.in_slot_bytes); }
            if (g.Co % 64 != 0) o.y_ptrs.clear();
            o.fo.resize(o.y_ptrs.size());
            for (size_t i = 0; i < o.y_ptrs.size(); ++i) ok = ok && tc::make_map_out(&o.fo[i], o.y_ptrs[i], g.Co, g.Wo, g.Ho, g.N, wt, ht);
            const bool pairs = c->kernel_path == 0;          // CTA-pair kernels for the 256-column tile (kernel_path 2: none)
            if (pairs && (o.n_tile_f >= 256 || (rows_ok && o.n_tile_f == 128))) {
                o.fbh.resize(m.D);
                for (int v = 0; v < m.D; ++v) ok = ok && tc::make_map_2d(&o.fbh[v], wbig(c, m, v, o.w_off), Ktot, g.Co, 64, o.n_tile_f / 2);
            }
            // ---- input gradient: dx[n, h, w, :] = sum over taps (r, s) with (h + pad - r), (w + pad - s) divisible by
            // the stride of dy[n, (h + pad - r) / stride, (w + pad - s) / stride, :] . W[:, r, s, :].
            // One launch per parity class (h mod stride, w mod stride); the class's pixels form a dense grid of the
            // size of dy.  A = dy (dense boxes), B = Wt [C][taps * Co] with flipped taps, output strided into dx.
            o.dgrad_needs_zero = false;
            tc::KmParams& d = o.kd; d = f;
            d.kchunks = g.Co / 64; d.xs = 1; d.ntaps = 0; d.ncls = 0;
            d.Hd = g.H / g.stride; d.Wd = g.W / g.stride; d.Ho = g.H; d.Wo = g.W; d.Co = g.C; d.Cn = g.C; d.os = g.stride;
            for (int ph = 0; ph < g.stride; ++ph) for (int pw = 0; pw < g.stride; ++pw) {
                const int first = d.ntaps;
                for (int r = 0; r < g.R; ++r) for (int q = 0; q < g.R; ++q) {
                    int a = ph + g.pad - r, b = pw + g.pad - q;
                    if (a % g.stride != 0 || b % g.stride != 0) continue;
                    d.dh[d.ntaps] = a / g.stride; d.dw[d.ntaps] = b / g.stride;
                    d.koff[d.ntaps] = (taps - 1 - (r * g.R + q)) * g.Co;
                    ++d.ntaps;
                }
                if (d.ntaps == first) { o.dgrad_needs_zero = true; continue; }
                d.cls_tap0[d.ncls] = first; d.cls_oph[d.ncls] = ph; d.cls_opw[d.ncls] = pw; ++d.ncls;
                d.cls_tap0[d.ncls] = d.ntaps;
            }
            o.da.resize(o.dy_ptrs.size());
            for (size_t i = 0; i < o.dy_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.da[i], o.dy_ptrs[i], g.Co, g.Wo, g.Ho, g.N, 64, wt, ht, nt, 1);
            // the input gradient: the tensor's own gradient buffer, or a slot of the hand-off to the previous module;
            // only a stride-1 layer writes it densely (tile geometry of dy = tile geometry of dx)
            if (g.stride == 1 && g.C % 64 == 0) {
                if (ti.own_grad) o.dx_ptrs.push_back(m.gradpool + ti.goff);
                else if (o.in == 0 && kk > 0) for (int i = 0; i < 2; ++i) o.dx_ptrs.push_back(m.d2 + (size_t)i * m.in_slot_bytes);
            }
            o.dox.resize(o.dx_ptrs.size());
            for (size_t i = 0; i < o.dx_ptrs.size(); ++i) ok = ok && tc::make_map_out(&o.dox[i], o.dx_ptrs[i], g.C, g.W, g.H, g.N, wt, ht);
            if (rows_ok) {
                o.dar.resize(o.dy_ptrs.size());
                for (size_t i = 0; i < o.dy_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.dar[i], o.dy_ptrs[i], g.Co, g.Wo, g.Ho, g.N, 64, g.Wo, ht + 2, 1, 1);
            }
            o.db.resize(m.D);
            for (int v = 0; v < m.D; ++v) ok = ok && tc::make_map_2d(&o.db[v], wtslot(m, v, o.w_off), (long)taps * g.Co, g.C, 64, o.n_tile_d);
            if (pairs && (o.n_tile_d >= 256 || (rows_ok && o.n_tile_d == 128))) {
                o.dbh.resize(m.D);
                for (int v = 0; v < m.D; ++v) ok = ok && tc::make_map_2d(&o.dbh[v], wtslot(m, v, o.w_off), (long)taps * g.Co, g.C, 64, o.n_tile_d / 2);
            }
            // ---- weight gradient: 64-pixel boxes of x (shifted per tap) and of dy
            tc::pixel_tile(g.Ho, g.Wo, 64, &wt, &ht, &nt);
            tc::WgParams& w = o.kw; w = tc::WgParams{};
            w.Wt = wt; w.Ht = ht; w.Nt = nt; w.tiles_w = g.Wo / wt; w.tiles_h = g.Ho / ht; w.tiles_n = (g.N + nt - 1) / nt;
            w.ptiles = w.tiles_w * w.tiles_h * w.tiles_n;
            w.ptiles_per_split = (w.ptiles + o.wg_splits - 1) / o.wg_splits;
            w.kchunks = g.C / 64; w.row_blocks = taps * w.kchunks; w.xs = g.stride; w.Co = g.Co;
            for (int t = 0; t < taps; ++t) { w.dh[t] = t / g.R - g.pad; w.dw[t] = t % g.R - g.pad; }
            o.wx.resize(o.a_ptrs.size());
            for (size_t i = 0; i < o.a_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.wx[i], o.a_ptrs[i], g.C, g.W, g.H, g.N, 64, wt, ht, nt, g.stride);
            o.wdy.resize(o.dy_ptrs.size());
            for (size_t i = 0; i < o.dy_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.wdy[i], o.dy_ptrs[i], g.Co, g.Wo, g.Ho, g.N, 64, wt, ht, nt, 1);
            if (o.wgr_variant) {
                // contraction steps of 128 pixels: dy through the input-gradient kernel's activation map (o.da), x with two extra rows
                tc::pixel_tile(g.Ho, g.Wo, 128, &wt, &ht, &nt);
                tc::WgRowsParams& q = o.kwr; q = tc::WgRowsParams{};
                q.W = g.W; q.Ht = ht; q.Nt = nt; q.tiles_h = g.Ho / ht; q.tiles_n = (g.N + nt - 1) / nt; q.C = g.C; q.Co = g.Co;
                o.wxr.resize(o.a_ptrs.size());
                for (size_t i = 0; i < o.a_ptrs.size(); ++i) ok = ok && tc::make_map_4d(&o.wxr[i], o.a_ptrs[i], g.C, g.W, g.H, g.N, 64, g.W, ht + 2, nt, 1);
            }
            if (!ok) return false;
            c->any_tc = true;
        }
    }
    return true;
}

fdg_status reset_state(fdg_ctx* ctx) {
    // tags: everything -1 (empty); weight slot 0 carries version 0
    size_t n_tags = 0;
    for (Module& m : ctx->mod) n_tags += 2 * (size_t)(m.in_depth + m.D + 2 + m.D) + 4;
    std::vector<int64_t> h(n_tags, -1);
    size_t pos = 0;
    for (Module& m : ctx->mod) {
        pos += 2 * (size_t)(m.in_depth + m.D + 2);
        h[pos + 1] = 0;                      // weight slot 0: version 0
        pos += 2 * (size_t)m.D + 4;
    }
    CK(cudaMemcpy(ctx->tags, h.data(), n_tags * sizeof(int64_t), cudaMemcpyHostToDevice));
    CK(cudaDeviceSynchronize());
    ctx->t = 0;
    for (Module& m : ctx->mod) m.had_bwd = false;
    return FDG_OK;
}

// Reads the device error word (the caller has synchronised the stream it cares about).
fdg_status check_device_error(fdg_ctx* ctx) {
    if (!ctx->any_tc && ctx->dt != 1) return FDG_OK;
    int e = 0;
    CK(cudaMemcpy(&e, ctx->tc_err, sizeof(int), cudaMemcpyDeviceToHost));
    if (e) return fail(ctx, FDG_ERR_TIMEOUT, "a kernel gave up waiting on an mbarrier (code %d)", e);
    return FDG_OK;
}

fdg_status run_step(fdg_ctx* ctx, const void* inputs, const int32_t* labels, bool host_src, float* host_loss) {
    if (!ctx) return FDG_ERR_INVALID_ARG;
    if (!inputs || !labels) return fail(ctx, FDG_ERR_INVALID_ARG, "inputs and labels must not be NULL");
    if (!ctx->have_params) return fail(ctx, FDG_ERR_STATE, "fdg_set_params must be called before fdg_step");
    if (ctx->broken) return fail(ctx, FDG_ERR_STATE, "an earlier step failed after part of its work was enqueued; call fdg_set_params to start over");
    const int K = ctx->K;
    const int64_t t = ctx->t;
    // 1. dependencies on the neighbours' previous iteration (all waits first, so that no wait sees an
    //    event recorded for THIS iteration)
    if (!ctx->serial && t > 0)
        for (int kk = 0; kk < K; ++kk) {
            Module& m = ctx->mod[kk];
            CK(cudaStreamWaitEvent(m.fstream, m.done, 0));                                   // weights t; slots its forward overwrites
            if (kk > 0) CK(cudaStreamWaitEvent(m.fstream, ctx->mod[kk - 1].fdone, 0));       // its input
            if (kk > 0) CK(cudaStreamWaitEvent(m.stream, ctx->mod[kk - 1].done, 0));         // reader of the hand-off slot it overwrites
            if (kk + 1 < K) CK(cudaStreamWaitEvent(m.stream, ctx->mod[kk + 1].done, 0));     // the error gradient it consumes
        }
    // 2. module 1 "samples" the batch of iteration t: copy into its FIFO slot; labels into the label FIFO
    {
        Module& m0 = ctx->mod[0];
        cudaMemcpyKind kind = host_src ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
        CK(cudaMemcpyAsync(m0.in_ring + (size_t)(t % m0.in_depth) * m0.in_slot_bytes, inputs,
                           (size_t)ctx->M * m0.in_elems * ctx->esz, kind, m0.fstream));
        CK(cudaMemcpyAsync(ctx->labels + (size_t)(t % ctx->label_depth) * ctx->M, labels, (size_t)ctx->M * sizeof(int32_t), kind, m0.fstream));
        CK(cudaEventRecord(ctx->ingested, m0.fstream));
    }
    // 3. every module: forward on tau_f, backward on tau_b, update
    for (int kk = 0; kk < K; ++kk) {
        Module& m = ctx->mod[kk];
        const int64_t tau_f = t - kk;                         // t - k + 1
        const int64_t tau_b = t - 2 * (int64_t)K + kk + 2;    // t - 2K + k + 1
        const int64_t v_b = tau_b + kk;                       // t - 2K + 2k: the version the forward of tau_b used
        const bool lastm = kk == K - 1;
        CK(cudaEventRecord(m.ev0, m.stream));
        TagOps tg{};
        if (tau_f >= 0) {
            tg.rd_act = m.tag_in + 2 * (tau_f % m.in_depth);
            tg.rd_wfwd = m.tag_w + 2 * (t % m.D);
            tg.wr_stash = m.tag_stash + 2 * (tau_f % m.D);
            if (!lastm) { Module& n = ctx->mod[kk + 1]; tg.wr_out = n.tag_in + 2 * (tau_f % n.in_depth); }
        }
        if (kk == 0) tg.wr_in = m.tag_in + 2 * (t % m.in_depth);   // the ingest above filled this slot with batch t
        if (tau_b >= 0) {
            tg.rd_stash = m.tag_stash + 2 * (tau_b % m.D);
            tg.rd_wbwd = m.tag_w + 2 * (v_b % m.D);
            if (!lastm) tg.rd_grad = ctx->mod[kk + 1].tag_d2 + 2 * ((t - 1) & 1);
            if (kk > 0) tg.wr_grad = m.tag_d2 + 2 * (t & 1);
        }
        tg.wr_wnext = m.tag_w + 2 * ((t + 1) % m.D);
        tg.fwd_batch = tau_f >= 0 ? tau_f : -1; tg.bwd_batch = tau_b >= 0 ? tau_b : -1; tg.version_now = t;
        tg.trace = m.trace;
        tags_step(tg, m.stream);

        if (tau_f >= 0) for (int g = 0; g < m.groups; ++g) forward_module(ctx, kk, tau_f, t, g);
        CK(cudaEventRecord(m.fdone, m.fstream));
        if (lastm && m.fstream != m.stream) CK(cudaStreamWaitEvent(m.stream, m.fdone, 0));   // the last module back-propagates the batch it just forwarded
        if (lastm) {
            float* loss_slot = ctx->loss_ring + (t % 64);
            // one replica: dphi/dlogits / M, the mean over all samples.  One replica per worker: / B, worker s's own
            // gradient scale 1/per_worker_batch of Eq. dl_update (the mixing matrix does the averaging)
            const bool fused_head = m.ops.back().head && m.groups == 1;     // the forward pass above has computed loss and dlogits
            if (tau_f >= 0 && fused_head) CK(cudaEventRecord(ctx->loss_ready, m.fstream));
            else if (tau_f >= 0) softmax_ce(ctx->dt, ctx->logits, ctx->labels + (size_t)(tau_f % ctx->label_depth) * ctx->M, ctx->dlogits,
                                       loss_slot, ctx->M, ctx->classes, ctx->R > 1 ? 1.f / (float)ctx->B : 1.f / (float)ctx->M, m.stream);
            else fill_f32(loss_slot, NAN, 1, m.stream);
            if (!(tau_f >= 0 && fused_head)) CK(cudaEventRecord(ctx->loss_ready, m.stream));
        }
        if (tau_b >= 0) for (int g = 0; g < m.groups; ++g) backward_module(ctx, kk, tau_b, v_b, t, g);
        // Eq. dl_update with P = 11^T/N: w(t+1) = w(t) - lr * averaged gradient; also emits version t+1
        // (after the forward pass has read version t: with a one-slot ring the update overwrites it)
        if (!lastm && m.fstream != m.stream) CK(cudaStreamWaitEvent(m.stream, m.fdone, 0));
        if (tau_b >= 0 && m.wstream != m.stream) { CK(cudaEventRecord(m.wdone, m.wstream)); CK(cudaStreamWaitEvent(m.stream, m.wdone, 0)); }
        if (ctx->R > 1) {
            // Eq. dl_update (a), (b) with a general P: u_r = w_r - lr g_r, w_s(t+1) = sum_r P_sr u_r, all replicas in one pass
            mix_update(ctx->dt, m.master, tau_b >= 0 ? m.grad : nullptr, wslot(ctx, m, t + 1, 0), m.n_big, m.n_small, m.wslot_bytes, ctx->R, ctx->P_dev,
                       ctx->lr, m.stream);
        } else if (m.fused_update) {
            Scope sc(KC_SGD, 0.0, (double)npar(m) * (tau_b >= 0 ? 12.0 : 4.0) + 2.0 * m.n_big + 4.0 * m.n_small + 2.0 * m.n_big, m.stream);
            CK(tc::run_update_module(m.upd, m.master, m.grad, wslot(ctx, m, t + 1), wtslot(m, t + 1, 0), wsmall(ctx, m, t + 1, 0), ctx->lr, tau_b >= 0, m.stream));
        } else {
            sgd_update(ctx->dt, m.master, tau_b >= 0 ? m.grad : nullptr, wslot(ctx, m, t + 1), m.n_big, ctx->lr, m.stream);
            if (m.n_small)
                sgd_update(0, m.master + m.n_big, tau_b >= 0 ? m.grad + m.n_big : nullptr,
                           wsmall(ctx, m, t + 1, 0), m.n_small, ctx->lr, m.stream);
            emit_transposed_weights(ctx, m, t + 1);
        }
        m.had_bwd = tau_b >= 0;
        CK(cudaEventRecord(m.ev1, m.stream));
        CK(cudaEventRecord(m.done, m.stream));
    }
    CK(cudaGetLastError());
    ctx->t = t + 1;
    if (host_loss) {
        CK(cudaEventSynchronize(ctx->loss_ready));          // the loss only: the last module's backward pass and update go on
        float l = 0.f;
        CK(cudaMemcpy(&l, ctx->loss_ring + (t % 64), sizeof(float), cudaMemcpyDeviceToHost));
        fdg_status es = check_device_error(ctx);
        if (es != FDG_OK) return es;
        *host_loss = l;
    }
    return FDG_OK;
}

}  // namespace

extern "C" {

const char* fdg_last_error(const fdg_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

void fdg_destroy(fdg_ctx* ctx) {
    if (!ctx) return;
    cudaDeviceSynchronize();
    for (Module& m : ctx->mod) {
        if (m.done) cudaEventDestroy(m.done);
        if (m.fdone) cudaEventDestroy(m.fdone);
        if (m.wev) cudaEventDestroy(m.wev);
        if (m.wdone) cudaEventDestroy(m.wdone);
        if (m.ev0) cudaEventDestroy(m.ev0);
        if (m.ev1) cudaEventDestroy(m.ev1);
    }
    if (ctx->ingested) cudaEventDestroy(ctx->ingested);
    if (ctx->loss_ready) cudaEventDestroy(ctx->loss_ready);
    for (cudaStream_t s : ctx->owned) cudaStreamDestroy(s);
    for (void* p : ctx->blocks) ctx->alloc.free(p, ctx->alloc.user);
    delete ctx;
}

fdg_status fdg_create(const fdg_layer* layers, int32_t n_layers, const int32_t* split_points, int32_t K,
                      int32_t n_workers, int32_t per_worker_batch, float lr, const fdg_options* opt,
                      const fdg_allocator* alloc, fdg_ctx** out) {
    fdg_ctx* ctx = nullptr;     // errors before the context exists go to the thread-local message
    if (!layers || n_layers <= 0 || K < 1 || (K > 1 && !split_points) || n_workers < 1 || per_worker_batch < 1 || !opt || !out)
        return fail(nullptr, FDG_ERR_INVALID_ARG, "null pointer or non-positive size");
    if (opt->dtype != 0 && opt->dtype != 1) return fail(nullptr, FDG_ERR_INVALID_ARG, "dtype must be 0 (fp32) or 1 (bf16)");
    if (opt->in_h < 1 || opt->in_w < 1 || opt->in_c < 1 || opt->num_classes < 2) return fail(nullptr, FDG_ERR_INVALID_ARG, "bad input shape or class count");
    if (K > 64) return fail(nullptr, FDG_ERR_INVALID_ARG, "K > 64");
    for (int k = 0; k + 1 < K; ++k) {
        int prev = k ? split_points[k - 1] : 0;
        if (split_points[k] <= prev || split_points[k] >= n_layers) return fail(nullptr, FDG_ERR_BAD_SPLIT, "split points must be strictly increasing inside 1..n_layers-1");
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); return fail(nullptr, FDG_ERR_ARCH, "no CUDA device"); }
    int dev = 0; cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return fail(nullptr, FDG_ERR_CUDA, "cannot query the device");
    if (prop.major != 10) return fail(nullptr, FDG_ERR_ARCH, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);

    ctx = new fdg_ctx();
    ctx->K = K; ctx->n_workers = n_workers; ctx->B = per_worker_batch; ctx->M = n_workers * per_worker_batch;
    ctx->dt = opt->dtype; ctx->esz = opt->dtype ? 2 : 4; ctx->classes = opt->num_classes; ctx->serial = opt->serial;
    ctx->kernel_path = opt->kernel_path;
    // modules on streams of their own: grids for a third of the SMs, so that tensor-core kernels and memory-bound kernels
    // of different modules run side by side instead of one after the other (a streamed batch-norm kernel keeps 92 % of
    // its bandwidth on half of the SMs, a tensor-core kernel takes 1.6 times as long there, not twice).  Measured on a
    // B200, ResNet-18-shaped, 4 modules, 30 steps under the power cap: 5.05-5.12 ms per step for 37..74 SMs against
    // 5.3-5.5 for all 148; VGG-shaped 0.77 against 0.90.  One stream: nothing runs beside a kernel, all SMs.
    ctx->grid_sms = opt->grid_sms > 0 ? (opt->grid_sms < prop.multiProcessorCount ? opt->grid_sms : prop.multiProcessorCount)
                                      : (opt->serial ? prop.multiProcessorCount : (prop.multiProcessorCount + 2) / 3);
    ctx->R = 1; ctx->P_dev = nullptr;
    if (opt->mixing) {
        // general mixing matrix: one weight replica per worker, every layer runs once per worker on the plain FMA kernels
        if (n_workers > mix_max_replicas()) { delete ctx; return fail(nullptr, FDG_ERR_UNSUPPORTED, "a mixing matrix is supported for at most %d workers", mix_max_replicas()); }
        ctx->R = n_workers; ctx->kernel_path = 1;
        ctx->P.assign(opt->mixing, opt->mixing + (size_t)n_workers * n_workers);
        for (int i = 0; i < n_workers; ++i) {
            double row = 0.0;
            for (int j = 0; j < n_workers; ++j) { const double v = ctx->P[(size_t)i * n_workers + j]; if (!(v == v) || std::fabs(v) > 1e6) row = NAN; row += v; }
            if (!(std::fabs(row - 1.0) <= 1e-6)) { delete ctx; return fail(nullptr, FDG_ERR_INVALID_ARG, "row %d of the mixing matrix does not sum to 1", i); }
        }
    }
    ctx->in_h = opt->in_h; ctx->in_w = opt->in_w; ctx->in_c = opt->in_c; ctx->lr = lr; ctx->t = 0; ctx->have_params = false; ctx->broken = false;
    ctx->layers.assign(layers, layers + n_layers);
    ctx->alloc = alloc ? *alloc : fdg_allocator{default_alloc, default_free, nullptr};
    ctx->own_streams = opt->streams == nullptr;
    ctx->device_bytes = 0;
    ctx->ingested = nullptr;
    ctx->loss_ready = nullptr;
    ctx->mod.resize(K);
    auto bail = [&](fdg_status s, const std::string& msg) { g_create_error = msg; fdg_destroy(ctx); return s; };

    int h = opt->in_h, w = opt->in_w, c = opt->in_c;
    size_t canon = 0;
    for (int kk = 0; kk < K; ++kk) {
        Module& m = ctx->mod[kk];
        m = Module{};
        m.p = kk ? split_points[kk - 1] : 0; m.q = kk + 1 < K ? split_points[kk] : n_layers;
        m.D = 2 * (K - kk - 1) + 1; m.in_depth = m.D + 2;
        std::string e = compile_module(ctx, m, h, w, c, kk == K - 1, canon);
        if (!e.empty()) {
            fdg_status s = e.rfind("BAD_SPLIT", 0) == 0 ? FDG_ERR_BAD_SPLIT : FDG_ERR_UNSUPPORTED;
            char buf[256]; snprintf(buf, sizeof buf, "module %d: %s", kk + 1, e.c_str());
            return bail(s, buf);
        }
        // worker groups (off unless asked for: measured slower on every configuration, see fdg_options.worker_groups):
        // a group is a whole number of workers; the last module of a split network stays whole
        m.groups = 1;
        if (ctx->R > 1) m.groups = n_workers;
        else if (opt->worker_groups > 1 && (kk + 1 < K || K == 1)) {
            int g = 1;
            while (g * 2 <= opt->worker_groups && n_workers % (g * 2) == 0) g *= 2;
            m.groups = g;
        }
        m.in_slot_bytes = align_up((size_t)ctx->M * m.in_elems * ctx->esz, 256);
        m.wslot_bytes = align_up(m.n_big * ctx->esz + m.n_small * sizeof(float), 256);
    }
    if (h * w * c != opt->num_classes) return bail(FDG_ERR_INVALID_ARG, "the last layer's width differs from num_classes");
    ctx->n_params = canon;
    ctx->label_depth = 2 * K;

    // ---- device memory
    bool oom = false;
    auto get = [&](size_t bytes) -> char* {
        if (oom) return nullptr;
        bytes = align_up(bytes ? bytes : 256, 256);
        void* p = ctx->alloc.alloc(bytes, ctx->alloc.user);
        if (!p) { oom = true; return nullptr; }
        ctx->blocks.push_back(p); ctx->device_bytes += bytes;
        return (char*)p;
    };
    size_t n_tags = 0;
    for (Module& m : ctx->mod) n_tags += 2 * (size_t)(m.in_depth + m.D + 2 + m.D) + 4;
    ctx->tags = (int64_t*)get(n_tags * sizeof(int64_t));
    ctx->labels = (int32_t*)get((size_t)ctx->label_depth * ctx->M * sizeof(int32_t));
    ctx->logits = (float*)get((size_t)ctx->M * ctx->classes * sizeof(float));
    ctx->dlogits = get((size_t)ctx->M * ctx->classes * ctx->esz);
    ctx->loss_ring = (float*)get(64 * sizeof(float));
    ctx->tc_err = (int*)get(256);
    if (ctx->R > 1) ctx->P_dev = (float*)get((size_t)ctx->R * ctx->R * sizeof(float));
    size_t tpos = 0;
    for (int kk = 0; kk < K && !oom; ++kk) {
        Module& m = ctx->mod[kk];
        m.in_ring = get((size_t)m.in_depth * m.in_slot_bytes);
        m.stash = get((size_t)m.D * m.stash_slot_bytes);
        m.gradpool = get(m.grad_pool_bytes);
        m.d2 = kk > 0 ? get(2 * m.in_slot_bytes) : nullptr;
        m.wring = get((size_t)m.D * ctx->R * m.wslot_bytes);
        m.wtring = (ctx->dt == 1 && ctx->R == 1) ? get((size_t)m.D * m.n_big * 2) : nullptr;
        m.master = (float*)get((size_t)ctx->R * (m.n_big + m.n_small) * sizeof(float));
        m.grad = (float*)get((size_t)ctx->R * (m.n_big + m.n_small) * sizeof(float));
        m.ws = (float*)get(m.ws_elems * sizeof(float));
        m.scratch = (float*)get(m.scratch_elems * sizeof(float));
        m.red = (float*)get(m.red_elems * sizeof(float));
        m.scratch_f = (float*)get(m.scratch_elems * sizeof(float));
        m.fwd_ws = m.fwd_ws_elems ? (float*)get(m.fwd_ws_elems * sizeof(float)) : nullptr;
        m.head_scratch = m.head_elems ? (float*)get(m.head_elems * sizeof(float)) : nullptr;
        m.cstat = m.cstat_elems ? (float*)get(m.cstat_elems * sizeof(float)) : nullptr;
        if (oom) break;
        m.tag_in = ctx->tags + tpos; tpos += 2 * (size_t)m.in_depth;
        m.tag_stash = ctx->tags + tpos; tpos += 2 * (size_t)m.D;
        m.tag_d2 = ctx->tags + tpos; tpos += 4;
        m.tag_w = ctx->tags + tpos; tpos += 2 * (size_t)m.D;
        m.trace = ctx->tags + tpos; tpos += 4;
    }
    if (oom) return bail(FDG_ERR_OOM, "the allocator returned NULL");
    // All streams have the same priority.  Measured on the ResNet-18-shaped benchmark: the step is bound by the sum of its
    // kernels, not by one module's chain, and ranking the later modules' short kernels first lengthened the first
    // module's step (the one with the largest tensors) by more than it saved elsewhere (5.65 against 5.50 ms per step).
    for (int kk = 0; kk < K; ++kk) {
        Module& m = ctx->mod[kk];
        cudaError_t e = cudaSuccess;
        if (opt->streams) m.stream = (cudaStream_t)opt->streams[ctx->serial ? 0 : kk];
        else if (ctx->serial && kk > 0) m.stream = ctx->mod[0].stream;
        else { e = cudaStreamCreateWithFlags(&m.stream, cudaStreamNonBlocking); if (e == cudaSuccess) ctx->owned.push_back(m.stream); }
        m.fstream = m.stream;
        if (e == cudaSuccess && !ctx->serial) { e = cudaStreamCreateWithFlags(&m.fstream, cudaStreamNonBlocking); if (e == cudaSuccess) ctx->owned.push_back(m.fstream); }
        m.wstream = m.stream;
        if (e == cudaSuccess && !ctx->serial) { e = cudaStreamCreateWithFlags(&m.wstream, cudaStreamNonBlocking); if (e == cudaSuccess) ctx->owned.push_back(m.wstream); }
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.wev, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.wdone, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.done, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&m.fdone, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreate(&m.ev0);
        if (e == cudaSuccess) e = cudaEventCreate(&m.ev1);
        if (e == cudaSuccess) e = cudaMemset(m.grad, 0, (size_t)ctx->R * (m.n_big + m.n_small) * sizeof(float));
        if (e == cudaSuccess) e = cudaMemset(m.master, 0, (size_t)ctx->R * (m.n_big + m.n_small) * sizeof(float));
        if (e != cudaSuccess) return bail(FDG_ERR_CUDA, cudaGetErrorString(e));
    }
    if (cudaEventCreateWithFlags(&ctx->ingested, cudaEventDisableTiming) != cudaSuccess) return bail(FDG_ERR_CUDA, "cudaEventCreate failed");
    if (cudaEventCreateWithFlags(&ctx->loss_ready, cudaEventDisableTiming) != cudaSuccess) return bail(FDG_ERR_CUDA, "cudaEventCreate failed");
    if (cudaMemset(ctx->tc_err, 0, 256) != cudaSuccess) return bail(FDG_ERR_CUDA, "cudaMemset failed");
    if (ctx->R > 1) {
        std::vector<float> pf(ctx->P.begin(), ctx->P.end());
        if (cudaMemcpy(ctx->P_dev, pf.data(), pf.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) return bail(FDG_ERR_CUDA, "cudaMemcpy failed");
    }
    ctx->any_tc = false;
    if (!build_tc_plans(ctx)) return bail(FDG_ERR_CUDA, "cuTensorMapEncodeTiled rejected a tensor map");
    // a group must hold whole image tiles of every tensor-core tiling: a ragged tile would reach into the next group's rows
    for (Module& m : ctx->mod) {
        const int n = ctx->M / m.groups;
        for (const Op& o : m.ops)
            if (o.tc && (n % o.kf.Nt || (o.kd.Nt && n % o.kd.Nt) || n % o.kw.Nt)) m.groups = 1;
    }
    // modules whose update runs as one kernel (instead of two update launches and one transposing launch per tensor-core
    // layer): bf16, one weight copy, all workers at once, at least one tensor-core layer
    for (Module& m : ctx->mod) {
        m.fused_update = false;
        tc::UpdTable& tb = m.upd; tb = tc::UpdTable{};
        if (ctx->dt != 1 || ctx->R != 1 || m.groups != 1) continue;
        size_t pos = 0;                              // everything below pos is covered
        bool fits = true;
        auto plain = [&](size_t a, size_t b) { if (b > a) { if (tb.nranges < 14) tb.ranges[tb.nranges++] = tc::UpdRange{a, b - a}; else fits = false; } };
        for (const Op& o : m.ops) {
            if (o.type != OP_CONV || !o.tc) continue;
            if (tb.nops == 12) { fits = false; break; }
            const int taps = o.g.R * o.g.R;
            plain(pos, o.w_off);
            tc::UpdOp u{}; u.w_off = o.w_off; u.Co = o.g.Co; u.taps = taps; u.Ci = o.g.C; u.tile0 = tb.total_tiles;
            tb.total_tiles += (taps * o.g.C / 32) * (o.g.Co / 32);
            tb.ops[tb.nops++] = u;
            pos = o.w_off + (size_t)taps * o.g.C * o.g.Co;
        }
        plain(pos, npar(m));
        tb.n_big = m.n_big;
        m.fused_update = fits && tb.nops > 0;
    }
    *out = ctx;
    return FDG_OK;
}

fdg_status fdg_wait_ingest(fdg_ctx* ctx) {
    if (!ctx) return FDG_ERR_INVALID_ARG;
    if (ctx->t > 0) CK(cudaEventSynchronize(ctx->ingested));
    return FDG_OK;
}

fdg_status fdg_join(fdg_ctx* ctx, void* stream) {
    if (!ctx) return FDG_ERR_INVALID_ARG;
    if (ctx->t > 0)
        for (Module& m : ctx->mod) CK(cudaStreamWaitEvent((cudaStream_t)stream, m.done, 0));
    return FDG_OK;
}

fdg_status fdg_grid_sms(const fdg_ctx* ctx, int32_t* sms) {
    if (!ctx || !sms) return FDG_ERR_INVALID_ARG;
    *sms = ctx->grid_sms;
    return FDG_OK;
}

fdg_status fdg_param_count(const fdg_ctx* ctx, size_t* count) {
    if (!ctx || !count) return FDG_ERR_INVALID_ARG;
    *count = ctx->n_params;
    return FDG_OK;
}

fdg_status fdg_param_layout(const fdg_ctx* ctx, fdg_param_tensor* out, int32_t capacity, int32_t* count) {
    if (!ctx || !count || (out && capacity < 0)) return FDG_ERR_INVALID_ARG;
    int32_t n = 0;
    uint64_t off = 0;
    int module = 0;
    auto emit = [&](int layer, int role, int ndim, int64_t d0, int64_t d1, int64_t d2, int64_t d3) {
        const uint64_t cnt = (uint64_t)(d0 * d1 * d2 * d3);
        if (out && n < capacity) out[n] = fdg_param_tensor{layer, module, role, ndim, {d0, d1, d2, d3}, off, cnt};
        off += cnt; ++n;
    };
    for (int l = 0; l < (int)ctx->layers.size(); ++l) {
        while (module + 1 < ctx->K && l >= ctx->mod[module + 1].p) ++module;
        const fdg_layer& Y = ctx->layers[l];
        switch (Y.kind) {
            case FDG_LINEAR:
                emit(l, FDG_PARAM_W, 2, Y.c_out, Y.c_in, 1, 1);
                if (Y.flags & 1) emit(l, FDG_PARAM_BIAS, 1, Y.c_out, 1, 1, 1);
                break;
            case FDG_CONV3X3: case FDG_CONV1X1: {
                const int r = Y.kind == FDG_CONV3X3 ? 3 : 1;
                emit(l, FDG_PARAM_W, 4, Y.c_out, r, r, Y.c_in);
                if (Y.flags & 1) emit(l, FDG_PARAM_BIAS, 1, Y.c_out, 1, 1, 1);
                break; }
            case FDG_BATCHNORM:
                emit(l, FDG_PARAM_GAMMA, 1, Y.c_in, 1, 1, 1);
                emit(l, FDG_PARAM_BETA, 1, Y.c_in, 1, 1, 1);
                break;
            case FDG_RES_ADD:
                if (Y.flags & 1) {
                    emit(l, FDG_PARAM_PROJ_W, 4, Y.c_out, 1, 1, Y.c_in);
                    emit(l, FDG_PARAM_PROJ_GAMMA, 1, Y.c_out, 1, 1, 1);
                    emit(l, FDG_PARAM_PROJ_BETA, 1, Y.c_out, 1, 1, 1);
                }
                break;
            default: break;
        }
    }
    *count = n;
    return FDG_OK;
}

// Copy a canonical parameter vector into replica `worker` (all replicas if worker < 0) and emit its version-0 copies.
static fdg_status load_replicas(fdg_ctx* ctx, const float* host_params, int worker) {
    for (Module& m : ctx->mod) {
        std::vector<float> h(npar(m), 0.f);
        for (const Segment& s : m.segs)
            std::memcpy(h.data() + (s.big ? 0 : m.n_big) + s.internal, host_params + s.canon, s.count * sizeof(float));
        for (int r = 0; r < ctx->R; ++r) {
            if (worker >= 0 && r != worker) continue;
            float* master = m.master + (size_t)r * npar(m);
            // in-stream copy, then wait: a plain cudaMemcpy from pageable memory may return before the DMA has
            // landed, and the module streams are non-blocking streams that do not order behind the default stream
            CK(cudaMemcpyAsync(master, h.data(), h.size() * sizeof(float), cudaMemcpyHostToDevice, m.stream));
            CK(cudaStreamSynchronize(m.stream));
            // version 0 into weight slot 0
            sgd_update(ctx->dt, master, nullptr, wslot(ctx, m, 0, r), m.n_big, 0.f, m.stream);
            if (m.n_small) sgd_update(0, master + m.n_big, nullptr, wsmall(ctx, m, 0, 0, r), m.n_small, 0.f, m.stream);
        }
        if (ctx->R == 1) emit_transposed_weights(ctx, m, 0);
        CK(cudaMemsetAsync(m.grad, 0, (size_t)ctx->R * npar(m) * sizeof(float), m.stream));
    }
    return FDG_OK;
}

fdg_status fdg_set_params(fdg_ctx* ctx, const float* host_params, size_t count) {
    if (!ctx || !host_params) return FDG_ERR_INVALID_ARG;
    if (count != ctx->n_params) return fail(ctx, FDG_ERR_INVALID_ARG, "expected %zu parameters, got %zu", ctx->n_params, count);
    CK(cudaDeviceSynchronize());
    fdg_status s = load_replicas(ctx, host_params, -1);
    if (s != FDG_OK) return s;
    s = reset_state(ctx);
    if (s != FDG_OK) return s;
    CK(cudaDeviceSynchronize());
    ctx->have_params = true;
    ctx->broken = false;
    return FDG_OK;
}

fdg_status fdg_set_params_worker(fdg_ctx* ctx, int32_t worker, const float* host_params, size_t count) {
    if (!ctx || !host_params) return FDG_ERR_INVALID_ARG;
    if (count != ctx->n_params) return fail(ctx, FDG_ERR_INVALID_ARG, "expected %zu parameters, got %zu", ctx->n_params, count);
    if (ctx->R == 1) return fail(ctx, FDG_ERR_STATE, "the context keeps one weight copy for all workers (no mixing matrix was given)");
    if (worker < 0 || worker >= ctx->R) return fail(ctx, FDG_ERR_INVALID_ARG, "worker %d out of range", worker);
    if (!ctx->have_params || ctx->t != 0) return fail(ctx, FDG_ERR_STATE, "fdg_set_params_worker replaces one replica of the initial weights: call it after fdg_set_params and before the first step");
    CK(cudaDeviceSynchronize());
    fdg_status s = load_replicas(ctx, host_params, worker);
    if (s != FDG_OK) return s;
    CK(cudaDeviceSynchronize());
    return FDG_OK;
}

// A CUDA error in the middle of a step leaves some of its kernels enqueued and the iteration counter where it was:
// the context then refuses further steps until fdg_set_params resets the FIFOs.
static fdg_status guarded_step(fdg_ctx* ctx, const void* inputs, const int32_t* labels, bool host_src, float* host_loss) {
    const fdg_status s = run_step(ctx, inputs, labels, host_src, host_loss);
    if (ctx && (s == FDG_ERR_CUDA || s == FDG_ERR_TIMEOUT)) ctx->broken = true;
    return s;
}
fdg_status fdg_step(fdg_ctx* ctx, const void* dev_inputs, const int32_t* dev_labels, float* host_loss_or_null) {
    return guarded_step(ctx, dev_inputs, dev_labels, false, host_loss_or_null);
}
fdg_status fdg_step_host(fdg_ctx* ctx, const void* host_inputs, const int32_t* host_labels, float* host_loss_or_null) {
    return guarded_step(ctx, host_inputs, host_labels, true, host_loss_or_null);
}

// worker < 0: the parameters of replica 0, or the gradient averaged over the replicas
static fdg_status gather(fdg_ctx* ctx, bool grads, int worker, float* host_out, size_t capacity, size_t* count) {
    if (!ctx || !host_out) return FDG_ERR_INVALID_ARG;
    if (capacity < ctx->n_params) return fail(ctx, FDG_ERR_INVALID_ARG, "capacity %zu < %zu parameters", capacity, ctx->n_params);
    if (worker >= ctx->n_workers) return fail(ctx, FDG_ERR_INVALID_ARG, "worker %d out of range", worker);
    CK(cudaDeviceSynchronize());
    { fdg_status es = check_device_error(ctx); if (es != FDG_OK) return es; }
    for (Module& m : ctx->mod) {
        const size_t n = npar(m);
        std::vector<float> h(n, 0.f);
        if (!grads || m.had_bwd) {
            if (grads && worker < 0 && ctx->R > 1) {
                // (1/N) sum_s g_{s,k}, accumulated in double
                std::vector<float> one(n);
                std::vector<double> acc(n, 0.0);
                for (int r = 0; r < ctx->R; ++r) {
                    CK(cudaMemcpy(one.data(), m.grad + (size_t)r * n, n * sizeof(float), cudaMemcpyDeviceToHost));
                    for (size_t i = 0; i < n; ++i) acc[i] += one[i];
                }
                for (size_t i = 0; i < n; ++i) h[i] = (float)(acc[i] / ctx->R);
            } else {
                const int r = (ctx->R > 1 && worker > 0) ? worker : 0;       // one copy: every worker has the same
                CK(cudaMemcpy(h.data(), (grads ? m.grad : m.master) + (size_t)r * n, n * sizeof(float), cudaMemcpyDeviceToHost));
            }
        }
        for (const Segment& s : m.segs)
            std::memcpy(host_out + s.canon, h.data() + (s.big ? 0 : m.n_big) + s.internal, s.count * sizeof(float));
    }
    if (count) *count = ctx->n_params;
    return FDG_OK;
}
fdg_status fdg_params(fdg_ctx* ctx, float* host_out, size_t capacity, size_t* count) { return gather(ctx, false, -1, host_out, capacity, count); }
fdg_status fdg_grads(fdg_ctx* ctx, float* host_out, size_t capacity, size_t* count) { return gather(ctx, true, -1, host_out, capacity, count); }
fdg_status fdg_params_worker(fdg_ctx* ctx, int32_t worker, float* host_out, size_t capacity, size_t* count) {
    if (worker < 0) return FDG_ERR_INVALID_ARG;
    return gather(ctx, false, worker, host_out, capacity, count);
}
fdg_status fdg_grads_worker(fdg_ctx* ctx, int32_t worker, float* host_out, size_t capacity, size_t* count) {
    if (worker < 0) return FDG_ERR_INVALID_ARG;
    if (ctx && ctx->R == 1) return fail(ctx, FDG_ERR_STATE, "the context keeps one averaged gradient (no mixing matrix was given)");
    return gather(ctx, true, worker, host_out, capacity, count);
}

// delta(t) = max over layers l and workers s of || w_{s,l}(t) - (1/N) sum_r w_{r,l}(t) ||_2   (Sec. 5, Eq. max_consensus_error)
fdg_status fdg_consensus_error(fdg_ctx* ctx, double* delta) {
    if (!ctx || !delta) return FDG_ERR_INVALID_ARG;
    if (ctx->R == 1) { *delta = 0.0; return FDG_OK; }       // one copy: the replicas cannot differ
    int32_t nt = 0;
    fdg_param_layout(ctx, nullptr, 0, &nt);
    std::vector<fdg_param_tensor> lay(nt);
    fdg_param_layout(ctx, lay.data(), nt, &nt);
    std::vector<std::vector<float>> w(ctx->R, std::vector<float>(ctx->n_params));
    for (int r = 0; r < ctx->R; ++r) {
        fdg_status s = gather(ctx, false, r, w[r].data(), ctx->n_params, nullptr);
        if (s != FDG_OK) return s;
    }
    double worst = 0.0;
    for (size_t i = 0; i < lay.size();) {
        size_t j = i;                                       // tensors i..j-1 belong to one layer
        while (j < lay.size() && lay[j].layer == lay[i].layer) ++j;
        const size_t a = lay[i].offset, b = lay[j - 1].offset + lay[j - 1].count;
        std::vector<double> mean(b - a, 0.0);
        for (int r = 0; r < ctx->R; ++r) for (size_t e = a; e < b; ++e) mean[e - a] += w[r][e];
        for (double& v : mean) v /= ctx->R;
        for (int r = 0; r < ctx->R; ++r) {
            double ss = 0.0;
            for (size_t e = a; e < b; ++e) { const double d = (double)w[r][e] - mean[e - a]; ss += d * d; }
            worst = std::max(worst, std::sqrt(ss));
        }
        i = j;
    }
    *delta = worst;
    return FDG_OK;
}

fdg_status fdg_trace(fdg_ctx* ctx, int64_t* fwd_batch, int64_t* bwd_batch, int64_t* bwd_weight_version, int32_t K) {
    if (!ctx || !fwd_batch || !bwd_batch || !bwd_weight_version || K != ctx->K) return FDG_ERR_INVALID_ARG;
    CK(cudaDeviceSynchronize());
    for (int kk = 0; kk < K; ++kk) {
        int64_t tr[4];
        CK(cudaMemcpy(tr, ctx->mod[kk].trace, sizeof tr, cudaMemcpyDeviceToHost));
        fwd_batch[kk] = tr[0];
        bwd_batch[kk] = tr[1]; bwd_weight_version[kk] = tr[2];
    }
    return FDG_OK;
}

fdg_status fdg_set_lr(fdg_ctx* ctx, float lr) {
    if (!ctx || !(lr >= 0.f)) return FDG_ERR_INVALID_ARG;
    ctx->lr = lr;
    return FDG_OK;
}

fdg_status fdg_stats(const fdg_ctx* ctx, size_t* device_bytes, uint64_t* kernel_launches) {
    if (!ctx) return FDG_ERR_INVALID_ARG;
    if (device_bytes) *device_bytes = ctx->device_bytes;
    if (kernel_launches) *kernel_launches = launches();
    return FDG_OK;
}

fdg_status fdg_profile(fdg_ctx* ctx, int32_t enable) {
    if (!ctx) return FDG_ERR_INVALID_ARG;
    CK(cudaDeviceSynchronize());
    profile_enable(enable != 0);
    return FDG_OK;
}

fdg_status fdg_profile_read(fdg_ctx* ctx, fdg_kernel_stat* out, int32_t capacity, int32_t* count) {
    if (!ctx || !out || !count) return FDG_ERR_INVALID_ARG;
    KernelStat st[KC_COUNT]; const char* names[KC_COUNT];
    int n = profile_read(st, names), w = 0;
    for (int i = 0; i < n && w < capacity; ++i) {
        if (!st[i].launches) continue;
        std::memset(&out[w], 0, sizeof out[w]);
        std::strncpy(out[w].name, names[i], sizeof(out[w].name) - 1);
        out[w].launches = st[i].launches; out[w].ms = st[i].ms; out[w].flops = st[i].flops; out[w].bytes = st[i].bytes;
        ++w;
    }
    // then the per-shape breakdown of the classes that carry a detail tag
    static KernelStat ds[192]; static char dn[192][48];
    int nd = profile_read_detail(ds, dn, 192);
    for (int i = 0; i < nd && w < capacity; ++i) {
        std::memset(&out[w], 0, sizeof out[w]);
        std::strncpy(out[w].name, dn[i], sizeof(out[w].name) - 1);
        out[w].launches = ds[i].launches; out[w].ms = ds[i].ms; out[w].flops = ds[i].flops; out[w].bytes = ds[i].bytes;
        ++w;
    }
    *count = w;
    return FDG_OK;
}

fdg_status fdg_module_times(fdg_ctx* ctx, float* ms, int32_t K) {
    if (!ctx || !ms || K != ctx->K) return FDG_ERR_INVALID_ARG;
    if (ctx->t == 0) return fail(ctx, FDG_ERR_STATE, "no step has run yet");
    CK(cudaDeviceSynchronize());
    for (int kk = 0; kk < K; ++kk) CK(cudaEventElapsedTime(&ms[kk], ctx->mod[kk].ev0, ctx->mod[kk].ev1));
    return FDG_OK;
}

}  // extern "C"
