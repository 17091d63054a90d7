// CPU ORACLE -- TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, fp64 implementation of one training iteration of a network split into K
// modules under fully decoupled parallel backpropagation combined with S data-parallel
// workers whose updates are mixed by a weight matrix P (paper Sec. 3.2, Sec. 3.3, update
// rule Eq. "dl_update" (a)/(b), Algorithm 1).  It exists to check the CUDA library and to be
// timed beside it.  It shares no code with the CUDA path and nothing in the product imports it.
//
// How it follows the paper:
//  * every agent (s,k) is simulated separately: own weights w_{s,k}, own inbox, own stash;
//  * the delay schedule is never computed from a closed form: an agent forwards whatever its
//    predecessor posted in the previous iteration and back-propagates whatever error gradient
//    its successor posted in the previous iteration (Algorithm 1's send/receive pairs);
//  * the backward pass of batch tau in module k uses the weights the forward pass of that batch
//    used (Sec. 3.2, backward pass: the module's own weights of version t-2K+2k), taken from the stash;
//  * u_{s,k} = w_{s,k} - eta * g_{s,k};  w_{s,k}(t+1) = sum_r P_{sr} u_{r,k}   (Eq. dl_update),
//    g = 0 while no error gradient has arrived (tau < 0);
//  * layers are the textbook definitions written as loops (Eq. forward_step / backward_step).
//
// Pins (tests/test_oracle_*.py): finite differences, torch-autograd on tiny nets, closed-form
// softmax/SGD cases, K=1 S=1 reduction to ordinary SGD, composite-weight identity
// (gradient of batch tau == plain backprop through col{w_k(tau+k-1)}), worker-average ==
// concatenated-batch gradient, brute-force recount of the schedule, matrix form of the mixing.
// Parity unpinned: none of the functions below; the paper's convergence theorems and its
// CIFAR-10 curves are not executed at all.
//
// Readings of the paper taken here (each is also listed in the design document):
//  * p_1 = 1 (layer 0 is the input); the message sent backwards is the gradient w.r.t. the
//    module's input; the mixing sum includes the agent itself (matrix form (P (x) I));
//  * loss = softmax cross-entropy (natural log); per-sample gradient scale c is a parameter
//    (c = 1/B with P = 11^T/S gives "SGD on the mean over all S*B samples");
//  * batch-norm: training mode, statistics per worker over its B*H*W values, biased variance,
//    eps = 1e-5; max-pool ties: first index in row-major window order; relu'(0) = 0.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <thread>
#include <vector>

namespace {

enum Kind { LINEAR = 0, CONV3X3, CONV1X1, RELU, MAXPOOL2, GLOBAL_AVGPOOL, BATCHNORM, RES_BEGIN, RES_ADD };
struct Layer { int32_t kind, c_in, c_out, stride, flags; };
constexpr double BN_EPS = 1e-5;

int g_threads = 0;   // 0 = hardware_concurrency
// Smallest distance of any value from a kink seen since the last reset: |x| at a ReLU, the gap
// between the two largest values of a max-pool window.  Tests use it to tell whether a lower
// precision could legitimately take the other branch somewhere.
double g_kink_margin = 1e300;
std::mutex g_kink_mu;
void note_kink(double m) { std::lock_guard<std::mutex> lk(g_kink_mu); g_kink_margin = std::min(g_kink_margin, m); }

int num_threads() {
    int n = g_threads > 0 ? g_threads : (int)std::thread::hardware_concurrency();
    return n < 1 ? 1 : n;
}

// Run fn(i) for i in [0,n) on up to `budget` threads (static interleaving); the outermost call's budget is
// num_threads().  A parallel_for reached from inside another one gets its share of the outer budget (the
// workers are the outer level; with fewer workers than threads the layer loops below use the rest).
// Every loop that is split this way writes disjoint outputs and keeps its own summation order, so the
// results do not depend on the number of threads.
thread_local int t_budget = 0;       // 0: outermost level
void parallel_for(int n, const std::function<void(int)>& fn) {
    const int budget = t_budget > 0 ? t_budget : num_threads();
    const int nt = std::min(budget, n);
    if (nt <= 1) { for (int i = 0; i < n; ++i) fn(i); return; }
    const int inner = std::max(1, budget / nt);
    std::vector<std::thread> th;
    for (int w = 0; w < nt; ++w)
        th.emplace_back([=, &fn] { t_budget = inner; for (int i = w; i < n; i += nt) fn(i); });
    for (auto& t : th) t.join();
}

struct Tensor {                       // [n, h, w, c], c fastest
    int n = 0, h = 0, w = 0, c = 0;
    std::vector<double> v;
    Tensor() = default;
    Tensor(int n_, int h_, int w_, int c_) : n(n_), h(h_), w(w_), c(c_), v((size_t)n_ * h_ * w_ * c_, 0.0) {}
    size_t per_sample() const { return (size_t)h * w * c; }
    double* at(int i, int y, int x) { return v.data() + (((size_t)i * h + y) * w + x) * c; }
    const double* at(int i, int y, int x) const { return v.data() + (((size_t)i * h + y) * w + x) * c; }
};

// ---- optional storage model of the bf16 configurations -------------------------------------
// "bf16 activations and weights with fp32 master weights and accumulation": arithmetic stays
// fp64 here, but every tensor the configuration STORES in bf16 is rounded when it is stored:
// value -> fp32 (round to nearest even) -> bf16 (round to nearest even).  Storage points:
//   forward : output of a linear/conv layer (after bias), of batch-norm (after the residual add
//             that directly follows it, if any), of the shortcut's projection conv and batch-norm,
//             of the residual add, of the pooling layers; NOT the logits of the last layer;
//             ReLU commutes with rounding, so it needs no point of its own;
//   weights : the matrices W (biases, gamma, beta stay unrounded);
//   backward: softmax-CE gradient, every input-gradient a layer hands on (a conv that opens a
//             residual block hands its gradient to the add unrounded; the sum is rounded once).
double round_bf16(double v) {
    float f = (float)v;
    uint32_t u; std::memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return f;              // inf / nan unchanged
    u += 0x7fffu + ((u >> 16) & 1u); u &= 0xffff0000u;
    std::memcpy(&f, &u, 4);
    return f;
}
template <class TensorT> void store(TensorT& t, bool q) { if (q) for (auto& e : t.v) e = round_bf16(e); }

size_t layer_param_count(const Layer& L) {
    switch (L.kind) {
        case LINEAR:  return (size_t)L.c_in * L.c_out + ((L.flags & 1) ? L.c_out : 0);
        case CONV3X3: return (size_t)9 * L.c_in * L.c_out + ((L.flags & 1) ? L.c_out : 0);
        case CONV1X1: return (size_t)L.c_in * L.c_out + ((L.flags & 1) ? L.c_out : 0);
        case BATCHNORM: return (size_t)2 * L.c_in;
        case RES_ADD: return (L.flags & 1) ? (size_t)L.c_in * L.c_out + 2 * (size_t)L.c_out : 0;
        default: return 0;
    }
}

// ---------------------------------------------------------------- layer definitions (Eq. forward_step)

// y[n,ho,wo,co] = b[co] + sum_{r,s,ci} x[n, ho*st + r - pad, wo*st + s - pad, ci] * W[co][r][s][ci]
Tensor conv_fwd(const Tensor& x, const double* W, const double* b, int cout, int R, int st, int pad) {
    int ho = (x.h + 2 * pad - R) / st + 1, wo = (x.w + 2 * pad - R) / st + 1;
    Tensor y(x.n, ho, wo, cout);
    int cin = x.c;
    parallel_for(x.n, [&](int i) {
        for (int oy = 0; oy < ho; ++oy) for (int ox = 0; ox < wo; ++ox) {
            double* yo = y.at(i, oy, ox);
            for (int co = 0; co < cout; ++co) {
                double acc = b ? b[co] : 0.0;
                for (int r = 0; r < R; ++r) {
                    int iy = oy * st + r - pad; if (iy < 0 || iy >= x.h) continue;
                    for (int s = 0; s < R; ++s) {
                        int ix = ox * st + s - pad; if (ix < 0 || ix >= x.w) continue;
                        const double* xi = x.at(i, iy, ix);
                        const double* wk = W + (((size_t)co * R + r) * R + s) * cin;
                        for (int ci = 0; ci < cin; ++ci) acc += xi[ci] * wk[ci];
                    }
                }
                yo[co] = acc;
            }
        }
    });
    return y;
}

// Chain rule for the convolution (Eq. backward_step): dX, dW (summed over the samples), db.
void conv_bwd(const Tensor& x, const Tensor& gy, const double* W, int R, int st, int pad,
              Tensor* gx, double* gW, double* gb) {
    int cin = x.c, cout = gy.c;
    if (gx) {
        *gx = Tensor(x.n, x.h, x.w, x.c);
        parallel_for(x.n, [&](int i) {
            for (int oy = 0; oy < gy.h; ++oy) for (int ox = 0; ox < gy.w; ++ox) {
                const double* g = gy.at(i, oy, ox);
                for (int r = 0; r < R; ++r) {
                    int iy = oy * st + r - pad; if (iy < 0 || iy >= x.h) continue;
                    for (int s = 0; s < R; ++s) {
                        int ix = ox * st + s - pad; if (ix < 0 || ix >= x.w) continue;
                        double* d = gx->at(i, iy, ix);
                        for (int co = 0; co < cout; ++co) {
                            const double* wk = W + (((size_t)co * R + r) * R + s) * cin;
                            double gv = g[co];
                            for (int ci = 0; ci < cin; ++ci) d[ci] += gv * wk[ci];
                        }
                    }
                }
            }
        });
    }
    parallel_for(cout, [&](int co) {            // one thread owns one output channel: no races
        double bsum = 0.0;
        for (int i = 0; i < x.n; ++i)
            for (int oy = 0; oy < gy.h; ++oy) for (int ox = 0; ox < gy.w; ++ox) {
                double gv = gy.at(i, oy, ox)[co];
                bsum += gv;
                for (int r = 0; r < R; ++r) {
                    int iy = oy * st + r - pad; if (iy < 0 || iy >= x.h) continue;
                    for (int s = 0; s < R; ++s) {
                        int ix = ox * st + s - pad; if (ix < 0 || ix >= x.w) continue;
                        const double* xi = x.at(i, iy, ix);
                        double* dw = gW + (((size_t)co * R + r) * R + s) * cin;
                        for (int ci = 0; ci < cin; ++ci) dw[ci] += gv * xi[ci];
                    }
                }
            }
        if (gb) gb[co] += bsum;
    });
}

// A linear layer is a 1x1 convolution over the flattened sample.
Tensor flatten(const Tensor& x) { Tensor y = x; y.c = (int)x.per_sample(); y.h = y.w = 1; return y; }

Tensor relu_fwd(const Tensor& x) {
    Tensor y = x;
    double margin = 1e300;
    for (auto& e : y.v) { margin = std::min(margin, std::fabs(e)); e = e > 0.0 ? e : 0.0; }
    note_kink(margin);
    return y;
}
Tensor relu_bwd(const Tensor& x, const Tensor& gy) {
    Tensor g = gy; for (size_t i = 0; i < g.v.size(); ++i) if (!(x.v[i] > 0.0)) g.v[i] = 0.0; return g;
}

Tensor maxpool_fwd(const Tensor& x) {
    Tensor y(x.n, x.h / 2, x.w / 2, x.c);
    double margin = 1e300;
    for (int i = 0; i < x.n; ++i) for (int oy = 0; oy < y.h; ++oy) for (int ox = 0; ox < y.w; ++ox)
        for (int c = 0; c < x.c; ++c) {
            double v[4] = {x.at(i, 2 * oy, 2 * ox)[c], x.at(i, 2 * oy, 2 * ox + 1)[c], x.at(i, 2 * oy + 1, 2 * ox)[c], x.at(i, 2 * oy + 1, 2 * ox + 1)[c]};
            double m = std::max(std::max(v[0], v[1]), std::max(v[2], v[3]));
            std::sort(v, v + 4);
            margin = std::min(margin, v[3] - v[2]);
            y.at(i, oy, ox)[c] = m;
        }
    note_kink(margin);
    return y;
}
Tensor maxpool_bwd(const Tensor& x, const Tensor& gy) {
    Tensor g(x.n, x.h, x.w, x.c);
    for (int i = 0; i < x.n; ++i) for (int oy = 0; oy < gy.h; ++oy) for (int ox = 0; ox < gy.w; ++ox)
        for (int c = 0; c < x.c; ++c) {
            int br = 0, bs = 0; double m = x.at(i, 2 * oy, 2 * ox)[c];
            for (int r = 0; r < 2; ++r) for (int s = 0; s < 2; ++s) {
                double v = x.at(i, 2 * oy + r, 2 * ox + s)[c];
                if (v > m) { m = v; br = r; bs = s; }          // strict: the first maximum wins
            }
            g.at(i, 2 * oy + br, 2 * ox + bs)[c] += gy.at(i, oy, ox)[c];
        }
    return g;
}

Tensor gap_fwd(const Tensor& x) {
    Tensor y(x.n, 1, 1, x.c);
    double inv = 1.0 / (x.h * x.w);
    for (int i = 0; i < x.n; ++i) for (int p = 0; p < x.h * x.w; ++p) for (int c = 0; c < x.c; ++c)
        y.v[(size_t)i * x.c + c] += x.v[((size_t)i * x.h * x.w + p) * x.c + c] * inv;
    return y;
}
Tensor gap_bwd(const Tensor& x, const Tensor& gy) {
    Tensor g(x.n, x.h, x.w, x.c);
    double inv = 1.0 / (x.h * x.w);
    for (int i = 0; i < x.n; ++i) for (int p = 0; p < x.h * x.w; ++p) for (int c = 0; c < x.c; ++c)
        g.v[((size_t)i * x.h * x.w + p) * x.c + c] = gy.v[(size_t)i * x.c + c] * inv;
    return g;
}

// Batch-norm over the whole tensor it is given (the caller passes ONE worker's batch).
struct BnSaved { std::vector<double> mean, invstd; };
Tensor bn_fwd(const Tensor& x, const double* gamma, const double* beta, BnSaved* sv) {
    int C = x.c; size_t N = x.v.size() / C;
    sv->mean.assign(C, 0.0); sv->invstd.assign(C, 0.0);
    for (size_t p = 0; p < N; ++p) for (int c = 0; c < C; ++c) sv->mean[c] += x.v[p * C + c];
    for (int c = 0; c < C; ++c) sv->mean[c] /= (double)N;
    std::vector<double> var(C, 0.0);
    for (size_t p = 0; p < N; ++p) for (int c = 0; c < C; ++c) { double d = x.v[p * C + c] - sv->mean[c]; var[c] += d * d; }
    for (int c = 0; c < C; ++c) sv->invstd[c] = 1.0 / std::sqrt(var[c] / (double)N + BN_EPS);
    Tensor y = x;
    for (size_t p = 0; p < N; ++p) for (int c = 0; c < C; ++c)
        y.v[p * C + c] = gamma[c] * (x.v[p * C + c] - sv->mean[c]) * sv->invstd[c] + beta[c];
    return y;
}
Tensor bn_bwd(const Tensor& x, const Tensor& gy, const double* gamma, const BnSaved& sv, double* ggamma, double* gbeta) {
    int C = x.c; size_t N = x.v.size() / C;
    std::vector<double> s1(C, 0.0), s2(C, 0.0);          // sum dy, sum dy * xhat
    for (size_t p = 0; p < N; ++p) for (int c = 0; c < C; ++c) {
        double xh = (x.v[p * C + c] - sv.mean[c]) * sv.invstd[c];
        s1[c] += gy.v[p * C + c]; s2[c] += gy.v[p * C + c] * xh;
    }
    Tensor g = x;
    for (size_t p = 0; p < N; ++p) for (int c = 0; c < C; ++c) {
        double xh = (x.v[p * C + c] - sv.mean[c]) * sv.invstd[c];
        g.v[p * C + c] = gamma[c] * sv.invstd[c] * (gy.v[p * C + c] - s1[c] / (double)N - xh * s2[c] / (double)N);
    }
    for (int c = 0; c < C; ++c) { ggamma[c] += s2[c]; gbeta[c] += s1[c]; }
    return g;
}

// Softmax cross-entropy per sample; returns the summed loss, writes scale * (softmax - onehot).
double softmax_ce(const Tensor& logits, const int32_t* labels, double scale, Tensor* g) {
    int C = logits.c; double total = 0.0;
    *g = Tensor(logits.n, 1, 1, C);
    for (int i = 0; i < logits.n; ++i) {
        const double* z = logits.v.data() + (size_t)i * C;
        double m = z[0]; for (int c = 1; c < C; ++c) m = std::max(m, z[c]);
        double se = 0.0; for (int c = 0; c < C; ++c) se += std::exp(z[c] - m);
        double lse = m + std::log(se);
        total += lse - z[labels[i]];
        for (int c = 0; c < C; ++c) g->v[(size_t)i * C + c] = scale * (std::exp(z[c] - lse) - (c == labels[i] ? 1.0 : 0.0));
    }
    return total;
}

// ---------------------------------------------------------------- a module = a contiguous layer group

struct Saved {                         // h~_k(tau): what the backward pass of the group needs
    std::vector<Tensor> in;            // input of every layer
    std::vector<BnSaved> bn;           // per layer (used by BATCHNORM and projecting RES_ADD)
    std::vector<Tensor> sc_in, sc_conv; // RES_ADD: block input, projection conv output
};

// Forward layers [p,q) on ONE worker's batch x with parameters `prm` (the group's slice).
Tensor group_forward(const std::vector<Layer>& L, int p, int q, const double* prm, const Tensor& x0, Saved* sv, bool sq = false) {
    int n = q - p;
    sv->in.assign(n, Tensor()); sv->bn.assign(n, BnSaved()); sv->sc_in.assign(n, Tensor()); sv->sc_conv.assign(n, Tensor());
    std::vector<Tensor> shortcut;
    Tensor x = x0;
    for (int l = p; l < q; ++l) {
        const Layer& Y = L[l]; int j = l - p;
        const double* w = prm;
        switch (Y.kind) {
            case LINEAR: { sv->in[j] = x; Tensor f = flatten(x);
                x = conv_fwd(f, w, (Y.flags & 1) ? w + (size_t)Y.c_in * Y.c_out : nullptr, Y.c_out, 1, 1, 0);
                store(x, sq && l + 1 < (int)L.size()); break; }
            case CONV3X3: sv->in[j] = x;
                x = conv_fwd(x, w, (Y.flags & 1) ? w + (size_t)9 * Y.c_in * Y.c_out : nullptr, Y.c_out, 3, Y.stride, 1);
                store(x, sq); break;
            case CONV1X1: sv->in[j] = x;
                x = conv_fwd(x, w, (Y.flags & 1) ? w + (size_t)Y.c_in * Y.c_out : nullptr, Y.c_out, 1, Y.stride, 0);
                store(x, sq); break;
            case RELU: sv->in[j] = x; x = relu_fwd(x); break;
            case MAXPOOL2: sv->in[j] = x; x = maxpool_fwd(x); break;
            case GLOBAL_AVGPOOL: sv->in[j] = x; x = gap_fwd(x); store(x, sq); break;
            case BATCHNORM: sv->in[j] = x; x = bn_fwd(x, w, w + Y.c_in, &sv->bn[j]);
                store(x, sq && !(l + 1 < q && L[l + 1].kind == RES_ADD)); break;
            case RES_BEGIN: shortcut.push_back(x); break;
            case RES_ADD: {
                Tensor s = shortcut.back(); shortcut.pop_back();
                sv->sc_in[j] = s;
                if (Y.flags & 1) {
                    Tensor cv = conv_fwd(s, w, nullptr, Y.c_out, 1, Y.stride, 0);
                    store(cv, sq);
                    sv->sc_conv[j] = cv;
                    const double* gb = w + (size_t)Y.c_in * Y.c_out;
                    s = bn_fwd(cv, gb, gb + Y.c_out, &sv->bn[j]);
                    store(s, sq);
                }
                for (size_t i = 0; i < x.v.size(); ++i) x.v[i] += s.v[i];
                store(x, sq);
                break; }
        }
        prm += layer_param_count(Y);
    }
    return x;
}

// Backward layers q-1..p with the SAME parameters the forward used; accumulates into gprm.
Tensor group_backward(const std::vector<Layer>& L, int p, int q, const double* prm, const Saved& sv,
                      const Tensor& gout, double* gprm, bool need_gin, bool sq = false) {
    std::vector<size_t> off(q - p + 1, 0);
    for (int l = p; l < q; ++l) off[l - p + 1] = off[l - p] + layer_param_count(L[l]);
    std::vector<Tensor> gshort;
    Tensor g = gout;
    for (int l = q - 1; l >= p; --l) {
        const Layer& Y = L[l]; int j = l - p;
        const double* w = prm + off[j]; double* gw = gprm + off[j];
        bool first = (l == p);                     // the group's first layer: input gradient optional
        switch (Y.kind) {
            case LINEAR: case CONV3X3: case CONV1X1: {
                int R = Y.kind == CONV3X3 ? 3 : 1, pad = Y.kind == CONV3X3 ? 1 : 0, st = Y.kind == LINEAR ? 1 : Y.stride;
                size_t nw = (size_t)R * R * Y.c_in * Y.c_out;
                Tensor gx; bool want = need_gin || !first;
                const Tensor& xs = sv.in[j];
                Tensor xin = Y.kind == LINEAR ? flatten(xs) : xs;
                conv_bwd(xin, g, w, R, st, pad, want ? &gx : nullptr, gw, (Y.flags & 1) ? gw + nw : nullptr);
                if (want) {
                    gx.h = xs.h; gx.w = xs.w; gx.c = xs.c; g = gx;               // undo the flattening
                    store(g, sq && !(l > p && L[l - 1].kind == RES_BEGIN));       // the add rounds the sum once
                }
                break; }
            case RELU: g = relu_bwd(sv.in[j], g); break;
            case MAXPOOL2: g = maxpool_bwd(sv.in[j], g); break;
            case GLOBAL_AVGPOOL: g = gap_bwd(sv.in[j], g); store(g, sq); break;
            case BATCHNORM: g = bn_bwd(sv.in[j], g, w, sv.bn[j], gw, gw + Y.c_in); store(g, sq); break;
            case RES_ADD: {
                Tensor gs = g;                     // d(a + s)/ds = 1
                if (Y.flags & 1) {
                    size_t nw = (size_t)Y.c_in * Y.c_out;
                    Tensor gc = bn_bwd(sv.sc_conv[j], gs, w + nw, sv.bn[j], gw + nw, gw + nw + Y.c_out);
                    store(gc, sq);
                    Tensor gx;
                    conv_bwd(sv.sc_in[j], gc, w, 1, Y.stride, 0, &gx, gw, nullptr);
                    store(gx, sq);
                    gs = gx;
                }
                gshort.push_back(gs);
                break; }
            case RES_BEGIN: {
                Tensor gs = gshort.back(); gshort.pop_back();
                for (size_t i = 0; i < g.v.size(); ++i) g.v[i] += gs.v[i];
                store(g, sq);
                break; }
        }
    }
    return g;
}

// ---------------------------------------------------------------- the S x K agents

struct Message { long batch = -1; Tensor t; std::vector<int32_t> labels; };
struct StashEntry { long version; std::vector<double> w; Saved sv; std::vector<int32_t> labels; Tensor out; };

struct Agent {
    std::vector<double> w;                         // w_{s,k}(t)
    Message act_in, act_next;                      // activation inbox: consumed now / posted for t+1
    Message grad_in, grad_next;                    // error-gradient inbox
    std::map<long, StashEntry> stash;
    std::vector<double> g;                         // g_{s,k} used in the last update
    size_t max_stash = 0;
};

struct Oracle {
    std::vector<Layer> layers;
    std::vector<int> first;                        // first[k] = p_k (0-based layer index), first[K] = L
    int K = 1, S = 1, B = 1, in_h = 1, in_w = 1, in_c = 1, classes = 10;
    double scale = 1.0;                            // c: per-sample gradient scale
    std::vector<double> P;                         // S x S mixing matrix
    bool use_current_weights = false;              // planted-mistake switch for tests
    bool storage_bf16 = false;                     // round at the storage points listed above
    long t = 0;
    std::vector<std::vector<Agent>> ag;            // [s][k]
    std::vector<size_t> poff;                      // parameter offset of module k in the full vector
    std::vector<long> tr_fwd, tr_bwd, tr_ver;      // last step's schedule, per module (from worker 0)
    double last_loss = NAN;
    long last_loss_batch = -1;
    std::string err;
};

size_t module_params(const Oracle& o, int k) { return o.poff[k + 1] - o.poff[k]; }

// The copy of a module's weights that the passes read: matrices rounded to bf16 when the storage
// model is on, everything else as it is.
std::vector<double> pass_weights(const Oracle& o, int p, int q, const std::vector<double>& w) {
    std::vector<double> c = w;
    if (!o.storage_bf16) return c;
    size_t off = 0;
    for (int l = p; l < q; ++l) {
        const Layer& Y = o.layers[l];
        size_t nmat = 0;
        if (Y.kind == LINEAR || Y.kind == CONV1X1) nmat = (size_t)Y.c_in * Y.c_out;
        else if (Y.kind == CONV3X3) nmat = (size_t)9 * Y.c_in * Y.c_out;
        else if (Y.kind == RES_ADD && (Y.flags & 1)) nmat = (size_t)Y.c_in * Y.c_out;
        for (size_t i = 0; i < nmat; ++i) c[off + i] = round_bf16(c[off + i]);
        off += layer_param_count(Y);
    }
    return c;
}

}  // namespace

extern "C" {

// layers: n_layers x 5 int32; splits: K-1 layer indices; P: S*S doubles (row-major) or NULL for 11^T/S.
void* orc_create(const int32_t* layers, int n_layers, const int32_t* splits, int K, int S, int B,
                 int in_h, int in_w, int in_c, int classes, const double* P, double grad_scale) {
    auto o = std::make_unique<Oracle>();
    o->layers.resize(n_layers);
    std::memcpy(o->layers.data(), layers, sizeof(Layer) * n_layers);
    o->K = K; o->S = S; o->B = B; o->in_h = in_h; o->in_w = in_w; o->in_c = in_c; o->classes = classes;
    o->scale = grad_scale;
    o->first.push_back(0);
    for (int k = 0; k + 1 < K; ++k) {
        if (splits[k] <= o->first.back() || splits[k] >= n_layers) return nullptr;
        o->first.push_back(splits[k]);
    }
    o->first.push_back(n_layers);
    o->poff.assign(K + 1, 0);
    for (int k = 0; k < K; ++k) {
        size_t c = 0; for (int l = o->first[k]; l < o->first[k + 1]; ++l) c += layer_param_count(o->layers[l]);
        o->poff[k + 1] = o->poff[k] + c;
    }
    o->P.assign((size_t)S * S, 1.0 / S);
    if (P) std::memcpy(o->P.data(), P, sizeof(double) * S * S);
    o->ag.assign(S, std::vector<Agent>(K));
    for (auto& row : o->ag) for (int k = 0; k < K; ++k) { row[k].w.assign(module_params(*o, k), 0.0); row[k].g.assign(module_params(*o, k), 0.0); }
    o->tr_fwd.assign(K, -1); o->tr_bwd.assign(K, -1); o->tr_ver.assign(K, -1);
    return o.release();
}
void orc_destroy(void* h) { delete (Oracle*)h; }
void orc_set_threads(int n) { g_threads = n; }
double orc_kink_margin(int reset) { double m = g_kink_margin; if (reset) g_kink_margin = 1e300; return m; }
int orc_threads() { return num_threads(); }
size_t orc_param_count(void* h) { return ((Oracle*)h)->poff.back(); }
void orc_set_flag_use_current_weights(void* h, int on) { ((Oracle*)h)->use_current_weights = on != 0; }
void orc_set_storage_bf16(void* h, int on) { ((Oracle*)h)->storage_bf16 = on != 0; }
void orc_round_bf16(const double* in, double* out, size_t n) { for (size_t i = 0; i < n; ++i) out[i] = round_bf16(in[i]); }

// worker < 0: set every replica to the same vector.
void orc_set_params(void* h, int worker, const double* p) {
    Oracle& o = *(Oracle*)h;
    for (int s = 0; s < o.S; ++s) if (worker < 0 || worker == s)
        for (int k = 0; k < o.K; ++k) std::copy(p + o.poff[k], p + o.poff[k + 1], o.ag[s][k].w.begin());
}
void orc_get_params(void* h, int worker, double* p) {
    Oracle& o = *(Oracle*)h;
    for (int k = 0; k < o.K; ++k) std::copy(o.ag[worker][k].w.begin(), o.ag[worker][k].w.end(), p + o.poff[k]);
}
// gradient g_{s,k} that entered the last update (zeros for modules that had no backward batch).
void orc_get_grads(void* h, int worker, double* p) {
    Oracle& o = *(Oracle*)h;
    for (int k = 0; k < o.K; ++k) std::copy(o.ag[worker][k].g.begin(), o.ag[worker][k].g.end(), p + o.poff[k]);
}
void orc_trace(void* h, int64_t* fwd, int64_t* bwd, int64_t* ver, int64_t* max_stash) {
    Oracle& o = *(Oracle*)h;
    for (int k = 0; k < o.K; ++k) { fwd[k] = o.tr_fwd[k]; bwd[k] = o.tr_bwd[k]; ver[k] = o.tr_ver[k]; max_stash[k] = (int64_t)o.ag[0][k].max_stash; }
}

// One iteration t of Algorithm 1 for all S*K agents.
// inputs: [S*B, in_h, in_w, in_c] doubles, worker-major; labels: [S*B]; eta: step size eta_t.
// loss_out: mean loss of the batch the last module processed in this iteration (NaN if none),
// loss_batch_out: its batch id.
int orc_step(void* h, const double* inputs, const int32_t* labels, double eta, double* loss_out, int64_t* loss_batch_out) {
    Oracle& o = *(Oracle*)h;
    const int K = o.K, S = o.S, B = o.B;
    const size_t in_per = (size_t)o.in_h * o.in_w * o.in_c;
    std::vector<double> loss_of(S, 0.0); std::vector<long> batch_of(S, -1);
    std::fill(o.tr_fwd.begin(), o.tr_fwd.end(), -1); std::fill(o.tr_bwd.begin(), o.tr_bwd.end(), -1); std::fill(o.tr_ver.begin(), o.tr_ver.end(), -1);

    // the data-groups are independent within an iteration (Algorithm 1: all agents in parallel)
    parallel_for(S, [&](int s) {
        double& loss_sum = loss_of[s]; long& loss_batch = batch_of[s];
        // agent (s,1) samples B_s(t): here, takes its rows of the caller's batch
        Message m; m.batch = o.t; m.t = Tensor(B, o.in_h, o.in_w, o.in_c);
        std::copy(inputs + (size_t)s * B * in_per, inputs + (size_t)(s + 1) * B * in_per, m.t.v.begin());
        m.labels.assign(labels + (size_t)s * B, labels + (size_t)(s + 1) * B);
        o.ag[s][0].act_in = std::move(m);

        for (int k = 0; k < K; ++k) {
            Agent& a = o.ag[s][k];
            const int p = o.first[k], q = o.first[k + 1];
            // ---- forward pass on whatever arrived (Algorithm 1: "compute h_l(t-k+1)")
            Tensor gout; long bwd_batch = -1;
            if (a.act_in.batch >= 0) {
                StashEntry e; e.version = o.t; e.w = pass_weights(o, p, q, a.w); e.labels = a.act_in.labels;
                Tensor out = group_forward(o.layers, p, q, e.w.data(), a.act_in.t, &e.sv, o.storage_bf16);
                if (s == 0) o.tr_fwd[k] = a.act_in.batch;
                if (k + 1 < K) {                       // send h_{q_k} to (s,k+1): it is read at t+1
                    Message nx; nx.batch = a.act_in.batch; nx.t = out; nx.labels = a.act_in.labels;
                    o.ag[s][k + 1].act_next = std::move(nx);
                } else {                               // last module: evaluate phi and its gradient
                    loss_sum += softmax_ce(out, e.labels.data(), o.scale, &gout);
                    store(gout, o.storage_bf16);
                    loss_batch = a.act_in.batch; bwd_batch = a.act_in.batch;
                }
                a.stash[a.act_in.batch] = std::move(e);
                a.max_stash = std::max(a.max_stash, a.stash.size());
                a.act_in = Message();
            }
            // ---- backward pass on the error gradient received from (s,k+1)
            if (k + 1 < K && a.grad_in.batch >= 0) { gout = a.grad_in.t; bwd_batch = a.grad_in.batch; a.grad_in = Message(); }
            std::fill(a.g.begin(), a.g.end(), 0.0);    // gradient is 0 while tau < 0
            if (bwd_batch >= 0) {
                StashEntry& e = a.stash.at(bwd_batch);
                const std::vector<double> wb = o.use_current_weights ? pass_weights(o, p, q, a.w) : e.w;
                Tensor gin = group_backward(o.layers, p, q, wb.data(), e.sv, gout, a.g.data(), k > 0, o.storage_bf16);
                if (s == 0) { o.tr_bwd[k] = bwd_batch; o.tr_ver[k] = e.version; }
                if (k > 0) {                           // send dphi/d(module input) to (s,k-1): read at t+1
                    Message nx; nx.batch = bwd_batch;
                    nx.t = gin;
                    o.ag[s][k - 1].grad_next = std::move(nx);
                }
                a.stash.erase(bwd_batch);
            }
        }
    });
    double loss_sum = 0.0; long loss_batch = -1;
    for (int s = 0; s < S; ++s) { loss_sum += loss_of[s]; loss_batch = std::max(loss_batch, batch_of[s]); }
    // ---- u_{s,k} = w_{s,k} - eta g_{s,k};  w_{s,k}(t+1) = sum_r P_sr u_{r,k}   (Eq. dl_update a, b)
    for (int k = 0; k < K; ++k) {
        size_t n = module_params(o, k);
        std::vector<std::vector<double>> u(S, std::vector<double>(n));
        for (int s = 0; s < S; ++s) for (size_t i = 0; i < n; ++i) u[s][i] = o.ag[s][k].w[i] - eta * o.ag[s][k].g[i];
        for (int s = 0; s < S; ++s) for (size_t i = 0; i < n; ++i) {
            double acc = 0.0; for (int r = 0; r < S; ++r) acc += o.P[(size_t)s * S + r] * u[r][i];
            o.ag[s][k].w[i] = acc;
        }
    }
    // ---- deliver the messages: what was sent in iteration t is received for iteration t+1
    for (int s = 0; s < S; ++s) for (int k = 0; k < K; ++k) {
        Agent& a = o.ag[s][k];
        if (a.act_next.batch >= 0) { a.act_in = std::move(a.act_next); a.act_next = Message(); }
        if (a.grad_next.batch >= 0) { a.grad_in = std::move(a.grad_next); a.grad_next = Message(); }
    }
    o.last_loss = loss_batch >= 0 ? loss_sum / ((double)S * B) : NAN;
    o.last_loss_batch = loss_batch;
    if (loss_out) *loss_out = o.last_loss;
    if (loss_batch_out) *loss_batch_out = loss_batch;
    o.t += 1;
    return 0;
}

// Ordinary (lock-step) backpropagation through the whole layer list with ONE parameter vector:
// loss = mean over the S*B samples; grad = scale * sum over samples of dphi/dW, batch-norm
// statistics per worker.  Used by tests for finite differences and the composite-weight identity.
double orc_plain_loss_grad(const int32_t* layers, int n_layers, int S, int B, int in_h, int in_w, int in_c,
                           const double* params, const double* inputs, const int32_t* labels,
                           double grad_scale, double* grad_or_null) {
    std::vector<Layer> L(n_layers); std::memcpy(L.data(), layers, sizeof(Layer) * n_layers);
    size_t np = 0; for (auto& y : L) np += layer_param_count(y);
    size_t in_per = (size_t)in_h * in_w * in_c;
    if (grad_or_null) std::fill(grad_or_null, grad_or_null + np, 0.0);
    double loss = 0.0;
    for (int s = 0; s < S; ++s) {
        Tensor x(B, in_h, in_w, in_c);
        std::copy(inputs + (size_t)s * B * in_per, inputs + (size_t)(s + 1) * B * in_per, x.v.begin());
        Saved sv; Tensor out = group_forward(L, 0, n_layers, params, x, &sv);
        Tensor g; loss += softmax_ce(out, labels + (size_t)s * B, grad_scale, &g);
        if (grad_or_null) group_backward(L, 0, n_layers, params, sv, g, grad_or_null, false);
    }
    return loss / ((double)S * B);
}

// Forward only: logits [S*B, classes] for tests.
void orc_plain_logits(const int32_t* layers, int n_layers, int S, int B, int in_h, int in_w, int in_c,
                      const double* params, const double* inputs, double* logits) {
    std::vector<Layer> L(n_layers); std::memcpy(L.data(), layers, sizeof(Layer) * n_layers);
    size_t in_per = (size_t)in_h * in_w * in_c;
    for (int s = 0; s < S; ++s) {
        Tensor x(B, in_h, in_w, in_c);
        std::copy(inputs + (size_t)s * B * in_per, inputs + (size_t)(s + 1) * B * in_per, x.v.begin());
        Saved sv; Tensor out = group_forward(L, 0, n_layers, params, x, &sv);
        std::copy(out.v.begin(), out.v.end(), logits + (size_t)s * B * out.per_sample());
    }
}

// Softmax cross-entropy alone (closed-form pins).
double orc_softmax_ce(const double* logits, const int32_t* labels, int n, int classes, double scale, double* grad) {
    Tensor z(n, 1, 1, classes); std::copy(logits, logits + (size_t)n * classes, z.v.begin());
    Tensor g; double l = softmax_ce(z, labels, scale, &g);
    std::copy(g.v.begin(), g.v.end(), grad);
    return l / n;
}

}  // extern "C"
