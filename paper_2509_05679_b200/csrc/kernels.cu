// Plain-FMA (CUDA-core) kernels: every layer kind in fp32 or bf16 storage with fp32 arithmetic.
// They are the whole fp32 path (true fp32 FMAs: TF32 would break the 1e-5 parameter tolerance)
// and, on the bf16 path, serve the shapes the tensor-core kernels do not take (3-channel stem,
// strided convs, 10-class head) plus all memory-bound elementwise / reduction work.
#include "kernels.h"

#include <cuda_bf16.h>
#include <atomic>
#include <cstdio>
#include <map>
#include <mutex>
#include <string>
#include <vector>

namespace fdg {

static std::atomic<uint64_t> g_launches{0};
uint64_t launches() { return g_launches.load(); }

// ---- per-kernel-class device timing (off by default): every launcher opens a Scope, which counts the
// launch and, while profiling is on, brackets it with two events on the launching stream.
static const char* kClassNames[KC_COUNT] = {
    "igemm_fma_fwd", "igemm_fma_dgrad", "igemm_fma_wgrad", "splitk_reduce", "bias_grad", "relu_fwd", "relu_bwd", "add_fwd",
    "copy_accumulate", "maxpool_fwd", "maxpool_bwd", "gap_fwd", "gap_bwd", "bn_fwd_stats", "bn_fwd_apply", "bn_bwd_reduce",
    "bn_bwd_apply", "softmax_ce", "sgd_update", "tags", "fill", "tc_gemm_fwd", "tc_gemm_dgrad", "tc_gemm_wgrad", "tc_aux"};
namespace prof {
struct Rec { int cls; cudaEvent_t a, b; };
static bool g_on = false;
static std::mutex g_mu;
static std::vector<Rec> g_recs;
static std::vector<cudaEvent_t> g_pool;
static KernelStat g_stat[KC_COUNT];
static std::map<std::string, KernelStat> g_detail;          // "class[detail]" -> statistics
static thread_local const char* t_detail = nullptr;
struct DRec { std::string key; cudaEvent_t a, b; };
static std::vector<DRec> g_drecs;
static cudaEvent_t get_event() {
    if (!g_pool.empty()) { cudaEvent_t e = g_pool.back(); g_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr; cudaEventCreate(&e); return e;
}
}  // namespace prof
void profile_detail(const char* d) { prof::t_detail = d; }
Scope::Scope(int cls_, double flops, double bytes, cudaStream_t s) : cls(cls_), st(s), a(nullptr), detail(prof::t_detail) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!prof::g_on) return;
    std::lock_guard<std::mutex> lk(prof::g_mu);
    prof::g_stat[cls].launches += 1; prof::g_stat[cls].flops += flops; prof::g_stat[cls].bytes += bytes;
    if (detail) {
        KernelStat& d = prof::g_detail[std::string(kClassNames[cls]) + "[" + detail + "]"];
        d.launches += 1; d.flops += flops; d.bytes += bytes;
    }
    a = prof::get_event();
    cudaEventRecord(a, st);
}
Scope::~Scope() {
    if (!a) return;
    std::lock_guard<std::mutex> lk(prof::g_mu);
    cudaEvent_t b = prof::get_event();
    cudaEventRecord(b, st);
    prof::g_recs.push_back({cls, a, b});
    if (detail) prof::g_drecs.push_back({std::string(kClassNames[cls]) + "[" + detail + "]", a, b});
}
void profile_enable(bool on) {
    std::lock_guard<std::mutex> lk(prof::g_mu);
    if (on) { for (auto& k : prof::g_stat) k = KernelStat{}; prof::g_detail.clear(); }
    prof::g_on = on;
}
int profile_read(KernelStat* out, const char** names) {
    cudaDeviceSynchronize();
    std::lock_guard<std::mutex> lk(prof::g_mu);
    for (auto& r : prof::g_drecs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) prof::g_detail[r.key].ms += ms;
    }
    prof::g_drecs.clear();
    for (auto& r : prof::g_recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) prof::g_stat[r.cls].ms += ms;
        prof::g_pool.push_back(r.a); prof::g_pool.push_back(r.b);
    }
    prof::g_recs.clear();
    for (int i = 0; i < KC_COUNT; ++i) { out[i] = prof::g_stat[i]; names[i] = kClassNames[i]; }
    return KC_COUNT;
}
int profile_read_detail(KernelStat* out, char (*names)[48], int capacity) {
    std::lock_guard<std::mutex> lk(prof::g_mu);
    int n = 0;
    for (auto& kv : prof::g_detail) {
        if (n >= capacity) break;
        out[n] = kv.second;
        std::snprintf(names[n], 48, "%s", kv.first.c_str());
        ++n;
    }
    return n;
}

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float ld(const float* p) { return *p; }
__device__ __forceinline__ float ld(const bf16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void st(float* p, float v) { *p = v; }
__device__ __forceinline__ void st(bf16* p, float v) { *p = __float2bfloat16_rn(v); }

static inline unsigned cdiv(size_t a, size_t b) { return (unsigned)((a + b - 1) / b); }

// ------------------------------------------------------------------------------------------
// Implicit GEMM  C[m][n] = sum_k A(m,k) * B(k,n)  with the operands gathered on the fly.
//   FWD  : m = output pixel, n = c_out, k = (r,s,c_in)
//   DGRAD: m = input pixel,  n = c_in,  k = (r,s,c_out)
//   WGRAD: m = c_out,        n = (r,s,c_in), k = output pixel   (split over blockIdx.z)
// 64x64 tile, 16-deep k slices, 256 threads, 4x4 outputs per thread.
// ------------------------------------------------------------------------------------------
enum { M_FWD = 0, M_DGRAD = 1, M_WGRAD = 2 };
constexpr int BM = 64, BN = 64, BK = 16;

template <typename T, int MODE>
__global__ void __launch_bounds__(256) igemm_simt(const T* __restrict__ P0, const T* __restrict__ P1,
                                                  void* __restrict__ out, const float* __restrict__ bias,
                                                  float* __restrict__ partial, ConvGeom g, int Mg, int Ng, int Kg,
                                                  int k_per_split, int epi) {
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int kbeg = blockIdx.z * k_per_split;
    const int kend = min(Kg, kbeg + k_per_split);

    // which element of the A / B tile this thread fetches: one row (column) and 4 consecutive k
    int a_row, a_kq, b_col, b_kq;
    if (MODE == M_WGRAD) { a_row = tid & 63; a_kq = tid >> 6; b_col = tid & 63; b_kq = tid >> 6; }
    else if (MODE == M_DGRAD) { a_row = tid >> 2; a_kq = tid & 3; b_col = tid & 63; b_kq = tid >> 6; }
    else { a_row = tid >> 2; a_kq = tid & 3; b_col = tid >> 2; b_kq = tid & 3; }

    const int HoWo = g.Ho * g.Wo, HW = g.H * g.W, RC = g.R * g.C, RCo = g.R * g.Co;
    const int am = m0 + a_row, bn = n0 + b_col;
    // per-thread decode of the fixed index
    int a_n = 0, a_y = 0, a_x = 0;       // FWD: (n, oy*st-pad, ox*st-pad); DGRAD: (n, iy+pad, ix+pad)
    if (MODE == M_FWD && am < Mg) { a_n = am / HoWo; int p = am - a_n * HoWo; int oy = p / g.Wo; a_y = oy * g.stride - g.pad; a_x = (p - oy * g.Wo) * g.stride - g.pad; }
    if (MODE == M_DGRAD && am < Mg) { a_n = am / HW; int p = am - a_n * HW; int iy = p / g.W; a_y = iy + g.pad; a_x = (p - iy * g.W) + g.pad; }
    int b_r = 0, b_s = 0, b_c = 0;       // WGRAD: n -> (r, s, ci)
    if (MODE == M_WGRAD && bn < Ng) { b_r = bn / RC; int q = bn - b_r * RC; b_s = q / g.C; b_c = q - b_s * g.C; }

    // acc + comp: compensated (Kahan) running sum of the per-slice partial sums, so that the rounding
    // error of a long contraction (3072 terms in the first MLP layer) stays at a few ulps
    float acc[4][4], comp[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; comp[i][j] = 0.f; }
    const int tx = tid & 15, ty = tid >> 4;

    for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // ---- A element
            int k = k0 + a_kq * 4 + j;
            float v = 0.f;
            if (am < Mg && k < kend) {
                if (MODE == M_FWD) {
                    int rs = k / g.C, ci = k - rs * g.C; int r = rs / g.R, s = rs - r * g.R;
                    int iy = a_y + r, ix = a_x + s;
                    if (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) v = ld(P0 + (((size_t)a_n * g.H + iy) * g.W + ix) * g.C + ci);
                } else if (MODE == M_DGRAD) {
                    int rs = k / g.Co, co = k - rs * g.Co; int r = rs / g.R, s = rs - r * g.R;
                    int ty_ = a_y - r, tx_ = a_x - s;
                    if (ty_ >= 0 && tx_ >= 0) {
                        int oy = ty_ / g.stride, ox = tx_ / g.stride;
                        if (oy * g.stride == ty_ && ox * g.stride == tx_ && oy < g.Ho && ox < g.Wo)
                            v = ld(P0 + (((size_t)a_n * g.Ho + oy) * g.Wo + ox) * g.Co + co);
                    }
                } else {
                    v = ld(P0 + (size_t)k * g.Co + am);
                }
            }
            As[a_kq * 4 + j][a_row] = v;
            // ---- B element
            k = k0 + b_kq * 4 + j;
            v = 0.f;
            if (bn < Ng && k < kend) {
                if (MODE == M_FWD) {
                    v = ld(P1 + (size_t)bn * Kg + k);
                } else if (MODE == M_DGRAD) {
                    int rs = k / g.Co, co = k - rs * g.Co;
                    v = ld(P1 + ((size_t)co * g.R * g.R + rs) * g.C + bn);
                } else {
                    int n = k / HoWo; int p = k - n * HoWo; int oy = p / g.Wo, ox = p - oy * g.Wo;
                    int iy = oy * g.stride - g.pad + b_r, ix = ox * g.stride - g.pad + b_s;
                    if (iy >= 0 && iy < g.H && ix >= 0 && ix < g.W) v = ld(P1 + (((size_t)n * g.H + iy) * g.W + ix) * g.C + b_c);
                }
            }
            Bs[b_kq * 4 + j][b_col] = v;
        }
        __syncthreads();
        float part[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) part[i][j] = 0.f;
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) part[i][j] = fmaf(a[i], b[j], part[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float y = part[i][j] - comp[i][j];
                float t = acc[i][j] + y;
                comp[i][j] = (t - acc[i][j]) - y;
                acc[i][j] = t;
            }
        __syncthreads();
    }
    (void)RCo;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= Mg) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n >= Ng) continue;
            size_t o = (size_t)m * Ng + n;
            float v = acc[i][j];
            if (partial) { partial[(size_t)blockIdx.z * Mg * Ng + o] = v; continue; }
            if (bias) v += bias[n];
            if (epi & EPI_RELU) v = fmaxf(v, 0.f);
            if (epi & EPI_OUT_F32) {
                float* c = (float*)out;
                c[o] = (epi & EPI_ACCUM) ? c[o] + v : v;
            } else {
                T* c = (T*)out;
                if (epi & EPI_ACCUM) v += ld(c + o);
                st(c + o, v);
            }
        }
    }
}

// out[i] = sum_z partial[z][i], z ascending (fixed order => run-to-run identical results)
__global__ void splitk_reduce(const float* __restrict__ partial, float* __restrict__ out, size_t n, int splits, bool accum) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int z = 0; z < splits; ++z) s += partial[(size_t)z * n + i];
    out[i] = accum ? out[i] + s : s;
}

void splitk_reduce_launch(const float* partial, float* out, size_t n, int splits, bool accum, cudaStream_t s) {
    Scope sc(KC_SPLITK, 0.0, 4.0 * n * (splits + 1), s);
    splitk_reduce<<<cdiv(n, 256), 256, 0, s>>>(partial, out, n, splits, accum);
}

int wgrad_splits(const ConvGeom& g) {
    long Kg = (long)g.N * g.Ho * g.Wo;
    int tiles = (int)(cdiv(g.Co, BM) * cdiv((size_t)g.R * g.R * g.C, BN));
    int want = (148 * 4 + tiles - 1) / tiles;               // about four waves of CTAs
    int maxs = (int)((Kg + 255) / 256);                     // at least 256 contraction rows per split
    int s = want < maxs ? want : maxs;
    if (s < 1) s = 1;
    if (s > 256) s = 256;
    return s;
}
size_t wgrad_workspace_elems(const ConvGeom& g) {
    int s = wgrad_splits(g);
    return s > 1 ? (size_t)s * g.Co * g.R * g.R * g.C : 0;
}

// out[m][n] = epilogue(sum_z partial[z][m][n] + bias[n]), z ascending
template <typename T>
__global__ void splitk_forward_epilogue(const float* __restrict__ partial, void* __restrict__ out, const float* __restrict__ bias, size_t n, int Ng, int splits, int epi) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float v = 0.f;
    for (int z = 0; z < splits; ++z) v += partial[(size_t)z * n + i];
    if (bias) v += bias[i % Ng];
    if (epi & EPI_RELU) v = fmaxf(v, 0.f);
    if (epi & EPI_OUT_F32) ((float*)out)[i] = v; else st((T*)out + i, v);
}
// A forward pass with few output tiles and a long contraction (a linear layer on a small batch: 8 CTAs walking 3072 terms)
// is split over the contraction so that it fills the GPU; the partial sums go through `ws`.
int forward_splits(const ConvGeom& g) {
    const long Mg = (long)g.N * g.Ho * g.Wo, Ng = g.Co, Kg = (long)g.R * g.R * g.C;
    const long tiles = (long)cdiv(Ng, BN) * cdiv(Mg, BM);
    if (tiles >= 74 || Kg < 512 || Mg * Ng > (1 << 18)) return 1;
    long s = (148 * 2) / tiles, maxs = Kg / 128;
    if (s > maxs) s = maxs;
    if (s > 32) s = 32;
    return (int)(s < 1 ? 1 : s);
}
size_t forward_workspace_elems(const ConvGeom& g) {
    const int s = forward_splits(g);
    return s > 1 ? (size_t)s * g.N * g.Ho * g.Wo * g.Co : 0;
}
template <typename T>
static void conv_forward_t(const void* x, const void* w, const float* bias, void* y, const ConvGeom& g, int epi, float* ws, size_t ws_elems, cudaStream_t s) {
    int Mg = g.N * g.Ho * g.Wo, Ng = g.Co, Kg = g.R * g.R * g.C;
    const double flops = 2.0 * Mg * Ng * Kg, bytes = sizeof(T) * ((double)g.N * g.H * g.W * g.C + (double)Ng * Kg + (double)Mg * Ng);
    int splits = ws ? forward_splits(g) : 1;
    while (splits > 1 && (size_t)splits * Mg * Ng > ws_elems) --splits;          // a window of the batch: stay inside the workspace sized for the whole batch
    if (splits > 1) {
        const int kps = ((Kg + splits - 1) / splits + BK - 1) / BK * BK;
        splits = (Kg + kps - 1) / kps;
        dim3 grid(cdiv(Ng, BN), cdiv(Mg, BM), splits);
        { Scope sc(KC_FMA_FWD, flops, bytes, s);
          igemm_simt<T, M_FWD><<<grid, 256, 0, s>>>((const T*)x, (const T*)w, nullptr, nullptr, ws, g, Mg, Ng, Kg, kps, 0); }
        Scope sc(KC_SPLITK, 0.0, 4.0 * (splits + 1) * Mg * Ng, s);
        splitk_forward_epilogue<T><<<cdiv((size_t)Mg * Ng, 256), 256, 0, s>>>(ws, y, bias, (size_t)Mg * Ng, Ng, splits, epi);
        return;
    }
    dim3 grid(cdiv(Ng, BN), cdiv(Mg, BM), 1);
    Scope sc(KC_FMA_FWD, flops, bytes, s);
    igemm_simt<T, M_FWD><<<grid, 256, 0, s>>>((const T*)x, (const T*)w, y, bias, nullptr, g, Mg, Ng, Kg, Kg, epi);
}
void conv_forward(int dt, const void* x, const void* w, const float* bias, void* y, const ConvGeom& g, int epi, float* ws, size_t ws_elems, cudaStream_t s) {
    if (dt) conv_forward_t<bf16>(x, w, bias, y, g, epi, ws, ws_elems, s); else conv_forward_t<float>(x, w, bias, y, g, epi, ws, ws_elems, s);
}

template <typename T>
static void conv_dgrad_t(const void* dy, const void* w, void* dx, const ConvGeom& g, int epi, cudaStream_t s) {
    int Mg = g.N * g.H * g.W, Ng = g.C, Kg = g.R * g.R * g.Co;
    dim3 grid(cdiv(Ng, BN), cdiv(Mg, BM), 1);
    Scope sc(KC_FMA_DGRAD, 2.0 * Mg * Ng * Kg, sizeof(T) * ((double)g.N * g.Ho * g.Wo * g.Co + (double)Ng * Kg + (double)Mg * Ng), s);
    igemm_simt<T, M_DGRAD><<<grid, 256, 0, s>>>((const T*)dy, (const T*)w, dx, nullptr, nullptr, g, Mg, Ng, Kg, Kg, epi);
}
void conv_dgrad(int dt, const void* dy, const void* w, void* dx, const ConvGeom& g, int epi, cudaStream_t s) {
    if (dt) conv_dgrad_t<bf16>(dy, w, dx, g, epi, s); else conv_dgrad_t<float>(dy, w, dx, g, epi, s);
}

template <typename T>
static void conv_wgrad_t(const void* x, const void* dy, float* dw, float* ws, const ConvGeom& g, bool accum, cudaStream_t s) {
    int Mg = g.Co, Ng = g.R * g.R * g.C, Kg = g.N * g.Ho * g.Wo;
    int splits = wgrad_splits(g);
    int kps = ((Kg + splits - 1) / splits + BK - 1) / BK * BK;
    splits = (Kg + kps - 1) / kps;
    dim3 grid(cdiv(Ng, BN), cdiv(Mg, BM), splits);
    double flops = 2.0 * Mg * Ng * Kg, bytes = sizeof(T) * ((double)g.N * g.H * g.W * g.C + (double)Kg * Mg) + 4.0 * Mg * Ng;
    if (splits == 1) {
        Scope sc(KC_FMA_WGRAD, flops, bytes, s);
        igemm_simt<T, M_WGRAD><<<grid, 256, 0, s>>>((const T*)dy, (const T*)x, dw, nullptr, nullptr, g, Mg, Ng, Kg, kps,
                                                   EPI_OUT_F32 | (accum ? EPI_ACCUM : 0));
    } else {
        { Scope sc(KC_FMA_WGRAD, flops, bytes, s);
          igemm_simt<T, M_WGRAD><<<grid, 256, 0, s>>>((const T*)dy, (const T*)x, dw, nullptr, ws, g, Mg, Ng, Kg, kps, EPI_OUT_F32); }
        splitk_reduce_launch(ws, dw, (size_t)Mg * Ng, splits, accum, s);
    }
}
void conv_wgrad(int dt, const void* x, const void* dy, float* dw, float* ws, const ConvGeom& g, bool accum, cudaStream_t s) {
    if (dt) conv_wgrad_t<bf16>(x, dy, dw, ws, g, accum, s); else conv_wgrad_t<float>(x, dy, dw, ws, g, accum, s);
}

// ------------------------------------------------------------------------------------------
// column sums (bias gradient): two stages, fixed order
// ------------------------------------------------------------------------------------------
constexpr int RED_CHUNKS = 64;

template <typename T>
__global__ void colsum_partial(const T* __restrict__ dy, float* __restrict__ part, long rows, int C) {
    int c = blockIdx.x * 32 + threadIdx.x;
    long per = (rows + gridDim.y - 1) / gridDim.y;
    long r0 = (long)blockIdx.y * per, r1 = min(rows, r0 + per);
    float s = 0.f;
    if (c < C) for (long r = r0 + threadIdx.y; r < r1; r += blockDim.y) s += ld(dy + r * C + c);
    __shared__ float sh[8][33];
    sh[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float t = 0.f;
        for (int i = 0; i < 8; ++i) t += sh[i][threadIdx.x];
        part[(size_t)blockIdx.y * C + c] = t;
    }
}
__global__ void colsum_final(const float* __restrict__ part, float* __restrict__ out, int chunks, int C, bool accum) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int i = 0; i < chunks; ++i) s += part[(size_t)i * C + c];
    out[c] = accum ? out[c] + s : s;
}
void bias_grad(int dt, const void* dy, float* db, float* scratch, long rows, int C, bool accum, cudaStream_t s) {
    int chunks = (int)(rows < RED_CHUNKS ? rows : RED_CHUNKS);
    dim3 grid(cdiv(C, 32), chunks), blk(32, 8);
    { Scope sc(KC_BIAS_GRAD, 0.0, (dt ? 2.0 : 4.0) * rows * C, s);
      if (dt) colsum_partial<bf16><<<grid, blk, 0, s>>>((const bf16*)dy, scratch, rows, C);
      else colsum_partial<float><<<grid, blk, 0, s>>>((const float*)dy, scratch, rows, C); }
    Scope sc(KC_BIAS_GRAD, 0.0, 4.0 * chunks * C, s);
    colsum_final<<<cdiv(C, 128), 128, 0, s>>>(scratch, db, chunks, C, accum);
}

// ------------------------------------------------------------------------------------------
// elementwise layers: 128-bit accesses (8 bf16 or 4 fp32 values per thread and pass), grid-stride loops over a grid of
// a few CTAs per SM; the last n % V elements are handled one by one by the first threads
// ------------------------------------------------------------------------------------------
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int V = 4;
    static __device__ __forceinline__ void load(const float* p, float (&f)[8]) { const float4 v = *(const float4*)p; f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    static __device__ __forceinline__ void store(float* p, const float (&f)[8]) { *(float4*)p = make_float4(f[0], f[1], f[2], f[3]); }
};
template <> struct Vec<bf16> {
    static constexpr int V = 8;
    static __device__ __forceinline__ void load(const bf16* p, float (&f)[8]) {
        const uint4 v = *(const uint4*)p; const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) { f[2 * j] = __uint_as_float(w[j] << 16); f[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u); }
    }
    static __device__ __forceinline__ void store(bf16* p, const float (&f)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { const __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]); w[j] = *(const uint32_t*)&t; }
        *(uint4*)p = make_uint4(w[0], w[1], w[2], w[3]);
    }
};
static unsigned ew_grid(size_t nvec) { size_t b = (nvec + 255) / 256; return (unsigned)(b < 1 ? 1 : (b > 148 * 8 ? 148 * 8 : b)); }

// OP 0: y = max(x, 0).  OP 1: dx (+)= dy * (y > 0)   (a = y, b = dy, o = dx).  OP 2: y = a + b.  OP 3: dst (+)= src   (a = src, o = dst).
template <typename T, int OP>
__global__ void __launch_bounds__(256) ew_k(const T* __restrict__ a, const T* __restrict__ b, T* o, size_t n, bool accum, bool aligned) {
    constexpr int V = Vec<T>::V;
    const size_t nvec = aligned ? n / V : 0, stride = (size_t)gridDim.x * blockDim.x, t0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = t0; i < nvec; i += stride) {
        float fa[8], fb[8], fo[8];
        Vec<T>::load(a + i * V, fa);
        if (OP == 1 || OP == 2) Vec<T>::load(b + i * V, fb);
        if ((OP == 1 || OP == 3) && accum) Vec<T>::load(o + i * V, fo);
#pragma unroll
        for (int j = 0; j < V; ++j) {
            float v;
            if (OP == 0) v = fmaxf(fa[j], 0.f);
            else if (OP == 1) v = fa[j] > 0.f ? fb[j] : 0.f;
            else if (OP == 2) v = fa[j] + fb[j];
            else v = fa[j];
            if ((OP == 1 || OP == 3) && accum) v += fo[j];
            fo[j] = v;
        }
        Vec<T>::store(o + i * V, fo);
    }
    for (size_t i = nvec * V + t0; i < n; i += stride) {
        float v;
        if (OP == 0) v = fmaxf(ld(a + i), 0.f);
        else if (OP == 1) v = ld(a + i) > 0.f ? ld(b + i) : 0.f;
        else if (OP == 2) v = ld(a + i) + ld(b + i);
        else v = ld(a + i);
        if ((OP == 1 || OP == 3) && accum) v += ld(o + i);
        st(o + i, v);
    }
}
template <int OP>
static void ew_launch(int dt, const void* a, const void* b, void* o, size_t n, bool accum, cudaStream_t s) {
    // a window of a tensor whose rows are no multiple of 16 bytes can start anywhere: such calls go element by element
    const bool aligned = (((uintptr_t)a | (uintptr_t)b | (uintptr_t)o) & 15) == 0;
    const size_t work = aligned ? n / (dt ? 8 : 4) : n;
    if (dt) ew_k<bf16, OP><<<ew_grid(work), 256, 0, s>>>((const bf16*)a, (const bf16*)b, (bf16*)o, n, accum, aligned);
    else ew_k<float, OP><<<ew_grid(work), 256, 0, s>>>((const float*)a, (const float*)b, (float*)o, n, accum, aligned);
}

void relu_forward(int dt, const void* x, void* y, size_t n, cudaStream_t s) {
    Scope sc(KC_RELU_FWD, 0.0, 2 * (dt ? 2.0 : 4.0) * n, s);
    ew_launch<0>(dt, x, nullptr, y, n, false, s);
}
void relu_backward(int dt, const void* y, const void* dy, void* dx, size_t n, bool accum, cudaStream_t s) {
    Scope sc(KC_RELU_BWD, 0.0, (accum ? 4 : 3) * (dt ? 2.0 : 4.0) * n, s);
    ew_launch<1>(dt, y, dy, dx, n, accum, s);
}
void add_forward(int dt, const void* a, const void* b, void* y, size_t n, cudaStream_t s) {
    Scope sc(KC_ADD_FWD, 0.0, 3 * (dt ? 2.0 : 4.0) * n, s);
    ew_launch<2>(dt, a, b, y, n, false, s);
}
void copy_or_accumulate(int dt, const void* src, void* dst, size_t n, bool accum, cudaStream_t s) {
    Scope sc(KC_COPY_ACC, 0.0, (accum ? 3 : 2) * (dt ? 2.0 : 4.0) * n, s);
    ew_launch<3>(dt, src, nullptr, dst, n, accum, s);
}

// ------------------------------------------------------------------------------------------
// Backward pass through "+ bias, ReLU" of a linear / conv layer in ONE pass over dy:  dy *= (y > 0) in place (if the layer
// has a ReLU) and db[c] = sum over rows of the masked dy (if it has a bias).  A thread keeps one 128-bit channel group for
// every row it visits; a CTA owns a contiguous row range; partial sums per CTA, then a fixed-order final sum.
// Used when C / V is a power of two <= 256 (V = 8 bf16 / 4 fp32 values per access); other widths take the generic kernels.
// ------------------------------------------------------------------------------------------
constexpr int RB_MAX_CHUNKS = 592;
template <typename T>
__global__ void __launch_bounds__(256) relu_bias_bwd_k(const T* __restrict__ y, T* dy, float* __restrict__ part, long rows, int C, long rows_per_cta) {
    constexpr int V = Vec<T>::V;
    const int cgs = C / V, rows_it = 256 / cgs, cg = threadIdx.x % cgs, rl = threadIdx.x / cgs;
    const long r0 = (long)blockIdx.x * rows_per_cta, r1 = min(rows, r0 + rows_per_cta);
    float s[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j] = 0.f;
    for (long r = r0 + rl; r < r1; r += rows_it) {
        const size_t o = (size_t)r * C + (size_t)cg * V;
        float g[8];
        Vec<T>::load(dy + o, g);
        if (y) {
            float a[8];
            Vec<T>::load(y + o, a);
#pragma unroll
            for (int j = 0; j < V; ++j) if (!(a[j] > 0.f)) g[j] = 0.f;
            Vec<T>::store(dy + o, g);
        }
#pragma unroll
        for (int j = 0; j < V; ++j) s[j] += g[j];
    }
    if (!part) return;
    __shared__ float sh[256][9];
#pragma unroll
    for (int j = 0; j < V; ++j) sh[threadIdx.x][j] = s[j];
    __syncthreads();
    for (int t = threadIdx.x; t < C; t += 256) {
        const int q = t / V, k = t % V;
        float acc = 0.f;
        for (int rr = 0; rr < rows_it; ++rr) acc += sh[rr * cgs + q][k];
        part[(size_t)blockIdx.x * C + t] = acc;
    }
}
// one warp per channel: lanes take the partials round-robin, then a fixed shuffle tree
__global__ void colsum_final_warp(const float* __restrict__ part, float* __restrict__ out, int chunks, int C, bool accum) {
    const int c = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (c >= C) return;
    float a = 0.f;
    for (int k = lane; k < chunks; k += 32) a += part[(size_t)k * C + c];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(0xffffffffu, a, d);
    if (lane == 0) out[c] = accum ? out[c] + a : a;
}
bool relu_bias_backward_supported(int dt, int C) {
    const int V = dt ? 8 : 4;
    if (C % V) return false;
    const int cgs = C / V;
    return cgs <= 256 && (cgs & (cgs - 1)) == 0;
}
size_t relu_bias_backward_scratch_elems(int C) { return (size_t)RB_MAX_CHUNKS * C; }
void relu_bias_backward(int dt, const void* y_or_null, void* dy, float* db_or_null, float* scratch, long rows, int C, bool accum, cudaStream_t s) {
    const int V = dt ? 8 : 4, rows_it = 256 / (C / V);
    long chunks = (rows + (long)rows_it * 8 - 1) / ((long)rows_it * 8);              // at least eight passes per CTA
    if (chunks > RB_MAX_CHUNKS) chunks = RB_MAX_CHUNKS;
    if (chunks < 1) chunks = 1;
    long per = (rows + chunks - 1) / chunks;
    per = (per + rows_it - 1) / rows_it * rows_it;
    chunks = (rows + per - 1) / per;
    const double esz = dt ? 2.0 : 4.0;
    { Scope sc(db_or_null ? KC_BIAS_GRAD : KC_RELU_BWD, 0.0, esz * rows * C * (y_or_null ? 3 : 1), s);
      if (dt) relu_bias_bwd_k<bf16><<<(unsigned)chunks, 256, 0, s>>>((const bf16*)y_or_null, (bf16*)dy, db_or_null ? scratch : nullptr, rows, C, per);
      else relu_bias_bwd_k<float><<<(unsigned)chunks, 256, 0, s>>>((const float*)y_or_null, (float*)dy, db_or_null ? scratch : nullptr, rows, C, per); }
    if (db_or_null) {
        Scope sc(KC_BIAS_GRAD, 0.0, 4.0 * chunks * C, s);
        colsum_final_warp<<<cdiv((size_t)C * 32, 256), 256, 0, s>>>(scratch, db_or_null, (int)chunks, C, accum);
    }
}

template <typename T>
__global__ void maxpool_fwd_k(const T* x, T* y, int N, int H, int W, int C) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    int Ho = H / 2, Wo = W / 2;
    size_t total = (size_t)N * Ho * Wo * C;
    if (i >= total) return;
    int c = i % C; size_t p = i / C; int ox = p % Wo; p /= Wo; int oy = p % Ho; int n = p / Ho;
    const T* b = x + (((size_t)n * H + 2 * oy) * W + 2 * ox) * C + c;
    float m = ld(b);
    m = fmaxf(m, ld(b + C)); m = fmaxf(m, ld(b + (size_t)W * C)); m = fmaxf(m, ld(b + (size_t)W * C + C));
    st(y + i, m);
}
template <typename T>
__global__ void maxpool_bwd_k(const T* x, const T* dy, T* dx, int N, int H, int W, int C, bool accum) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    int Ho = H / 2, Wo = W / 2;
    size_t total = (size_t)N * Ho * Wo * C;
    if (i >= total) return;
    int c = i % C; size_t p = i / C; int ox = p % Wo; p /= Wo; int oy = p % Ho; int n = p / Ho;
    size_t base = (((size_t)n * H + 2 * oy) * W + 2 * ox) * C + c;
    size_t o[4] = {base, base + (size_t)C, base + (size_t)W * C, base + (size_t)W * C + C};
    int best = 0; float m = ld(x + o[0]);
#pragma unroll
    for (int j = 1; j < 4; ++j) { float v = ld(x + o[j]); if (v > m) { m = v; best = j; } }   // first maximum wins
    float g = ld(dy + i);
#pragma unroll
    for (int j = 0; j < 4; ++j) { float v = (j == best) ? g : 0.f; if (accum) v += ld(dx + o[j]); st(dx + o[j], v); }
}
// the same with one 128-bit channel group per thread (C a multiple of the vector width)
template <typename T>
__global__ void __launch_bounds__(256) maxpool_fwd_vk(const T* __restrict__ x, T* __restrict__ y, int N, int H, int W, int C) {
    constexpr int V = Vec<T>::V;
    const int Ho = H / 2, Wo = W / 2, cgs = C / V;
    const size_t total = (size_t)N * Ho * Wo * cgs;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cg = (int)(i % cgs); size_t p = i / cgs; const int ox = (int)(p % Wo); p /= Wo; const int oy = (int)(p % Ho); const size_t n = p / Ho;
        const T* b = x + ((n * H + 2 * oy) * W + 2 * ox) * C + (size_t)cg * V;
        float a0[8], a1[8], a2[8], a3[8];
        Vec<T>::load(b, a0); Vec<T>::load(b + C, a1); Vec<T>::load(b + (size_t)W * C, a2); Vec<T>::load(b + (size_t)W * C + C, a3);
#pragma unroll
        for (int j = 0; j < V; ++j) a0[j] = fmaxf(fmaxf(a0[j], a1[j]), fmaxf(a2[j], a3[j]));
        Vec<T>::store(y + i * V, a0);
    }
}
template <typename T>
__global__ void __launch_bounds__(256) maxpool_bwd_vk(const T* __restrict__ x, const T* __restrict__ dy, T* dx, int N, int H, int W, int C, bool accum) {
    constexpr int V = Vec<T>::V;
    const int Ho = H / 2, Wo = W / 2, cgs = C / V;
    const size_t total = (size_t)N * Ho * Wo * cgs;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cg = (int)(i % cgs); size_t p = i / cgs; const int ox = (int)(p % Wo); p /= Wo; const int oy = (int)(p % Ho); const size_t n = p / Ho;
        const size_t base = ((n * H + 2 * oy) * W + 2 * ox) * C + (size_t)cg * V;
        const size_t o[4] = {base, base + (size_t)C, base + (size_t)W * C, base + (size_t)W * C + C};
        float a[4][8], g[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) Vec<T>::load(x + o[q], a[q]);
        Vec<T>::load(dy + i * V, g);
        int best[8];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            int b = 0; float m = a[0][j];
#pragma unroll
            for (int q = 1; q < 4; ++q) if (a[q][j] > m) { m = a[q][j]; b = q; }            // first maximum wins
            best[j] = b;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float v[8];
            if (accum) Vec<T>::load(dx + o[q], v);
#pragma unroll
            for (int j = 0; j < V; ++j) { const float t = best[j] == q ? g[j] : 0.f; v[j] = accum ? v[j] + t : t; }
            Vec<T>::store(dx + o[q], v);
        }
    }
}
void maxpool_forward(int dt, const void* x, void* y, int N, int H, int W, int C, cudaStream_t s) {
    const double esz_ = dt ? 2.0 : 4.0;
    Scope sc(KC_POOL_FWD, 0.0, 1.25 * esz_ * (double)N * H * W * C, s);
    size_t n = (size_t)N * (H / 2) * (W / 2) * C;
    if (C % (dt ? 8 : 4) == 0) {
        if (dt) maxpool_fwd_vk<bf16><<<ew_grid(n / 8), 256, 0, s>>>((const bf16*)x, (bf16*)y, N, H, W, C);
        else maxpool_fwd_vk<float><<<ew_grid(n / 4), 256, 0, s>>>((const float*)x, (float*)y, N, H, W, C);
        return;
    }
    if (dt) maxpool_fwd_k<bf16><<<cdiv(n, 256), 256, 0, s>>>((const bf16*)x, (bf16*)y, N, H, W, C);
    else maxpool_fwd_k<float><<<cdiv(n, 256), 256, 0, s>>>((const float*)x, (float*)y, N, H, W, C);
}
void maxpool_backward(int dt, const void* x, const void* dy, void* dx, int N, int H, int W, int C, bool accum, cudaStream_t s) {
    const double esz_ = dt ? 2.0 : 4.0;
    Scope sc(KC_POOL_BWD, 0.0, 2.25 * esz_ * (double)N * H * W * C, s);
    size_t n = (size_t)N * (H / 2) * (W / 2) * C;
    if (C % (dt ? 8 : 4) == 0) {
        if (dt) maxpool_bwd_vk<bf16><<<ew_grid(n / 8), 256, 0, s>>>((const bf16*)x, (const bf16*)dy, (bf16*)dx, N, H, W, C, accum);
        else maxpool_bwd_vk<float><<<ew_grid(n / 4), 256, 0, s>>>((const float*)x, (const float*)dy, (float*)dx, N, H, W, C, accum);
        return;
    }
    if (dt) maxpool_bwd_k<bf16><<<cdiv(n, 256), 256, 0, s>>>((const bf16*)x, (const bf16*)dy, (bf16*)dx, N, H, W, C, accum);
    else maxpool_bwd_k<float><<<cdiv(n, 256), 256, 0, s>>>((const float*)x, (const float*)dy, (float*)dx, N, H, W, C, accum);
}

template <typename T>
__global__ void gap_fwd_k(const T* x, T* y, int N, int HW, int C) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)N * C) return;
    int c = i % C; size_t n = i / C;
    float s = 0.f;
    for (int p = 0; p < HW; ++p) s += ld(x + (n * HW + p) * C + c);
    st(y + i, s / (float)HW);
}
template <typename T>
__global__ void gap_bwd_k(const T* dy, T* dx, int N, int HW, int C, bool accum) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)N * HW * C) return;
    int c = i % C; size_t n = i / ((size_t)HW * C);
    float v = ld(dy + n * C + c) / (float)HW;
    if (accum) v += ld(dx + i);
    st(dx + i, v);
}
// the same with one 16-byte vector (4 fp32 / 8 bf16 channels) per thread; C a multiple of the vector length
template <typename T>
__global__ void __launch_bounds__(256) gap_bwd_vk(const T* __restrict__ dy, T* __restrict__ dx, size_t nvec, int HW, int Cv, bool accum) {
    constexpr int V = Vec<T>::V;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += (size_t)gridDim.x * blockDim.x) {
        const int cv = (int)(i % Cv); const size_t n = i / ((size_t)HW * Cv);
        float g[8], o[8];
        Vec<T>::load(dy + (n * Cv + cv) * V, g);
        if (accum) Vec<T>::load(dx + i * V, o);
#pragma unroll
        for (int j = 0; j < V; ++j) g[j] = accum ? g[j] / (float)HW + o[j] : g[j] / (float)HW;
        Vec<T>::store(dx + i * V, g);
    }
}
void gap_forward(int dt, const void* x, void* y, int N, int HW, int C, cudaStream_t s) {
    const double esz_ = dt ? 2.0 : 4.0; (void)esz_;
    Scope sc(KC_GAP_FWD, 0.0, esz_ * (double)N * (HW + 1) * C, s);
    size_t n = (size_t)N * C;
    if (dt) gap_fwd_k<bf16><<<cdiv(n, 128), 128, 0, s>>>((const bf16*)x, (bf16*)y, N, HW, C);
    else gap_fwd_k<float><<<cdiv(n, 128), 128, 0, s>>>((const float*)x, (float*)y, N, HW, C);
    
}
void gap_backward(int dt, const void* dy, void* dx, int N, int HW, int C, bool accum, cudaStream_t s) {
    const double esz_ = dt ? 2.0 : 4.0; (void)esz_;
    Scope sc(KC_GAP_BWD, 0.0, esz_ * (double)N * (HW + 1) * C, s);
    size_t n = (size_t)N * HW * C;
    const int V = dt ? 8 : 4;
    if (C % V == 0 && ((uintptr_t)dy | (uintptr_t)dx) % 16 == 0) {
        const size_t nvec = n / V;
        if (dt) gap_bwd_vk<bf16><<<ew_grid(nvec), 256, 0, s>>>((const bf16*)dy, (bf16*)dx, nvec, HW, C / V, accum);
        else gap_bwd_vk<float><<<ew_grid(nvec), 256, 0, s>>>((const float*)dy, (float*)dx, nvec, HW, C / V, accum);
        return;
    }
    if (dt) gap_bwd_k<bf16><<<cdiv(n, 256), 256, 0, s>>>((const bf16*)dy, (bf16*)dx, N, HW, C, accum);
    else gap_bwd_k<float><<<cdiv(n, 256), 256, 0, s>>>((const float*)dy, (float*)dx, N, HW, C, accum);
    
}

// ------------------------------------------------------------------------------------------
// batch-norm, statistics per worker
// ------------------------------------------------------------------------------------------
// grid (C/32, chunks, workers), block (32, 8).  part: [chunk][worker][C][2]
template <typename T, bool BWD>
__global__ void bn_reduce_partial(const T* __restrict__ x, const T* __restrict__ out, const T* __restrict__ dout,
                                  const float* __restrict__ stats, float* __restrict__ part, long rpw, int C, bool relu) {
    int c = blockIdx.x * 32 + threadIdx.x;
    int w = blockIdx.z, nw = gridDim.z;
    long per = (rpw + gridDim.y - 1) / gridDim.y;
    long r0 = (long)blockIdx.y * per, r1 = min(rpw, r0 + per);
    float s1 = 0.f, s2 = 0.f;
    if (c < C) {
        float mean = 0.f, istd = 0.f;
        if (BWD) { mean = stats[((size_t)w * C + c) * 2]; istd = stats[((size_t)w * C + c) * 2 + 1]; }
        const float pivot = BWD ? 0.f : ld(x + (size_t)w * rpw * C + c);
        for (long r = r0 + threadIdx.y; r < r1; r += blockDim.y) {
            size_t o = ((size_t)w * rpw + r) * C + c;
            if (BWD) {
                float dy = ld(dout + o);
                if (relu && !(ld(out + o) > 0.f)) dy = 0.f;
                s1 += dy; s2 += dy * (ld(x + o) - mean) * istd;
            } else {
                // sums of (x - pivot): the pivot (the worker's first value of the channel) keeps the variance
                // formula E[d^2] - E[d]^2 from cancelling when |mean| >> std
                float v = ld(x + o) - pivot; s1 += v; s2 += v * v;
            }
        }
    }
    __shared__ float sh1[8][33], sh2[8][33];
    sh1[threadIdx.y][threadIdx.x] = s1; sh2[threadIdx.y][threadIdx.x] = s2;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float a = 0.f, b = 0.f;
        for (int i = 0; i < 8; ++i) { a += sh1[i][threadIdx.x]; b += sh2[i][threadIdx.x]; }
        size_t o = (((size_t)blockIdx.y * nw + w) * C + c) * 2;
        part[o] = a; part[o + 1] = b;
    }
}
// forward: stats[w][c] = (mean, invstd).  One thread per (w, c).
template <typename T>
__global__ void bn_stats_final(const float* __restrict__ part, const T* __restrict__ x, float* __restrict__ stats, int chunks, int nwC,
                               int C, long rpw) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nwC) return;
    double s1 = 0.0, s2 = 0.0;
    for (int k = 0; k < chunks; ++k) { s1 += part[((size_t)k * nwC + i) * 2]; s2 += part[((size_t)k * nwC + i) * 2 + 1]; }
    const int w = i / C, c = i - w * C;
    const double pivot = (double)ld(x + (size_t)w * rpw * C + c);       // the partial sums are sums of (x - pivot)
    double dm = s1 / (double)rpw, var = s2 / (double)rpw - dm * dm;
    if (var < 0.0) var = 0.0;
    stats[(size_t)i * 2] = (float)(pivot + dm);
    stats[(size_t)i * 2 + 1] = (float)(1.0 / sqrt(var + 1e-5));
}
// backward: red[w][c] = (sum dy, sum dy xhat); dgamma[c] = sum_w red[w][c].y; dbeta[c] = sum_w red[w][c].x
__global__ void bn_bwd_final(const float* __restrict__ part, float* __restrict__ red, float* __restrict__ dgamma,
                             float* __restrict__ dbeta, int chunks, int nw, int C, bool accum) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float g = 0.f, b = 0.f;
    for (int w = 0; w < nw; ++w) {
        float s1 = 0.f, s2 = 0.f;
        for (int k = 0; k < chunks; ++k) { size_t o = (((size_t)k * nw + w) * C + c) * 2; s1 += part[o]; s2 += part[o + 1]; }
        red[((size_t)w * C + c) * 2] = s1; red[((size_t)w * C + c) * 2 + 1] = s2;
        b += s1; g += s2;
    }
    dgamma[c] = accum ? dgamma[c] + g : g; dbeta[c] = accum ? dbeta[c] + b : b;
}
template <typename T>
__global__ void bn_apply_k(const T* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                           const T* __restrict__ res, T* __restrict__ y, const float* __restrict__ stats,
                           long rpw, int C, size_t total, bool relu) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int c = i % C; size_t row = i / C; int w = (int)(row / rpw);
    float mean = stats[((size_t)w * C + c) * 2], istd = stats[((size_t)w * C + c) * 2 + 1];
    float v = gamma[c] * (ld(x + i) - mean) * istd + beta[c];
    if (res) v += ld(res + i);
    if (relu) v = fmaxf(v, 0.f);
    st(y + i, v);
}
template <typename T>
__global__ void bn_bwd_apply_k(const T* __restrict__ x, const T* __restrict__ out, const T* __restrict__ dout,
                               const float* __restrict__ gamma, const float* __restrict__ stats, const float* __restrict__ red,
                               T* __restrict__ dx, bool accum_dx, T* __restrict__ dres, bool accum_dres,
                               long rpw, int C, size_t total, bool relu) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int c = i % C; size_t row = i / C; int w = (int)(row / rpw);
    size_t so = ((size_t)w * C + c) * 2;
    float mean = stats[so], istd = stats[so + 1];
    float dy = ld(dout + i);
    if (relu && !(ld(out + i) > 0.f)) dy = 0.f;
    float xh = (ld(x + i) - mean) * istd;
    float inv_n = 1.f / (float)rpw;
    float v = gamma[c] * istd * (dy - red[so] * inv_n - xh * red[so + 1] * inv_n);
    if (accum_dx) v += ld(dx + i);
    st(dx + i, v);
    if (dres) { float r = dy; if (accum_dres) r += ld(dres + i); st(dres + i, r); }
}

// ------------------------------------------------------------------------------------------
// Batch-norm, bf16 storage, streamed: a CTA owns a contiguous range of one worker's rows, which is one
// contiguous range of memory (NHWC).  One thread feeds a ring of shared-memory stages with bulk asynchronous
// copies (cp.async.bulk, completion on an mbarrier), 16 KB per input tensor and stage, so that about 90 KB per
// CTA are in flight whatever the registers hold; all 256 threads read 16-byte vectors (8 channels) from the
// stage, and results go straight to global memory.  A thread keeps the same 8 channels for every row.
// grid = (row chunks, workers).  Used when C/8 is a power of two <= 256.
// ------------------------------------------------------------------------------------------
constexpr int BNV_THREADS = 256;
constexpr int BNV_MAX_CHUNKS = 128;
constexpr int BV = 8;                               // channels per thread (one 128-bit access)
// ring geometry: the best of the measured family (rings of 48..192 KB, 1..4 CTAs per SM, tiles of 8..32 KB)
constexpr int BNS_TILE = 16384;                     // bytes per input tensor and stage
constexpr int BNS_CTAS = 2;                         // CTAs per SM the ring size allows
constexpr int BNS_RING = 96 * 1024;                 // shared memory of the ring (stages = tiles in the ring / input tensors, at most 8)
constexpr int BNS_VPT = BNS_TILE / 16 / 256;        // 16-byte vectors per thread and tile
constexpr long long BNS_WAIT_CYCLES = 4000000000LL; // ~2 s

constexpr int BP = BV / 2;                          // channel pairs per thread
__device__ __forceinline__ void unpack8(const uint4& v, float2 (&f)[BP]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < BP; ++j) f[j] = make_float2(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xffff0000u));
}
// round to nearest even; RELU: negative values become zero in the same conversion
template <bool RELU>
__device__ __forceinline__ uint4 pack8(const float2 (&f)[BP]) {
    uint32_t w[BP];
#pragma unroll
    for (int j = 0; j < BP; ++j) {
        if (RELU) asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(w[j]) : "f"(f[j].y), "f"(f[j].x));
        else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[j]) : "f"(f[j].y), "f"(f[j].x));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
// the one expression both passes use for the normalised value, so that the backward pass can recompute the sign of
// the forward output from x alone: gamma * ((x - mean) * invstd) + beta, the product rounded before the fused last
// step, two channels per instruction
__device__ __forceinline__ float2 bn_pair(float2 x, float2 neg_mean, float2 invstd, float2 gamma, float2 beta) {
    return __ffma2_rn(gamma, __fmul2_rn(__fadd2_rn(x, neg_mean), invstd), beta);
}

__device__ __forceinline__ uint32_t bns_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bns_wait(uint32_t bar, uint32_t parity, int* err) {
    uint32_t ok;
    long long t0 = 0;
    for (;;) {
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (t0 == 0) t0 = clock64();
        else if (clock64() - t0 > BNS_WAIT_CYCLES) { atomicCAS(err, 0, 20); return false; }
    }
}

// p[0] + p[stride] + ... (n terms, in that order), eight loads in flight
__device__ __forceinline__ float2 sum_strided(const float2* p, size_t stride, int n) {
    float2 acc = make_float2(0.f, 0.f);
    int i = 0;
    for (; i + 8 <= n; i += 8) {
        float2 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = p[(size_t)(i + j) * stride];
#pragma unroll
        for (int j = 0; j < 8; ++j) { acc.x += v[j].x; acc.y += v[j].y; }
    }
    for (; i < n; ++i) { const float2 v = p[(size_t)i * stride]; acc.x += v.x; acc.y += v.y; }
    return acc;
}
// a fixed shuffle tree: the summation order never changes
__device__ __forceinline__ float2 warp_sum2(float2 v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) { v.x += __shfl_xor_sync(0xffffffffu, v.x, d); v.y += __shfl_xor_sync(0xffffffffu, v.y, d); }
    return v;
}

struct BnsArgs {
    const bf16* in[3];          // input tensors streamed through the ring: x, then dout, then the forward output (as the mode needs)
    int n_in;
    const float* gamma; const float* beta; const float* stats; const bf16* res;
    float* part;                // modes 0, 1: partial sums [chunk][worker][C][2], written; mode 3: the same, read (gridDim.x chunks)
    float* dgamma; float* dbeta; int accum_params;   // mode 3: parameter gradients, written by one CTA
    bf16* y;                    // mode 2: output; mode 3: dx
    bf16* dres;                 // mode 3: gradient of the residual input, or nullptr
    long rpw; int C; int relu; int mask_from_x; int accum_dx; int accum_dres;
    int reverse;                // walk the CTA's tiles from the last to the first: a kernel that re-reads what the kernel before it
                                // has just streamed in ascending order (backward apply after backward sums) starts with the part
                                // that is still in L2
    int* err;
};

// MODE 0: (sum x, sum x^2).  MODE 1: (sum dy, sum dy * xhat) with dy = dout * [forward output > 0] if relu.
// MODE 2: y = bn(x) (+ res) (relu).  MODE 3: dx (+)= BN backward of dy, dres (+)= dy.
// mask_from_x: the forward output had no residual, so its sign is the sign of bn_pair(x).
template <int MODE>
__global__ void __launch_bounds__(BNV_THREADS, BNS_CTAS) bns_kernel(const BnsArgs a) {
    extern __shared__ __align__(128) uint8_t bns_sm[];
    const int C = a.C, cgs = C / BV, rows_it = BNV_THREADS / cgs;
    const int tid = threadIdx.x, cg = tid % cgs, rl = tid / cgs;
    const int w = blockIdx.y, nw = gridDim.y;
    const int n_in = a.n_in, stages = (BNS_RING / BNS_TILE) / n_in < 8 ? (BNS_RING / BNS_TILE) / n_in : 8;
    const int tile_rows = BNS_TILE / (C * 2);
    long per = (a.rpw + gridDim.x - 1) / gridDim.x;
    per = (per + tile_rows - 1) / tile_rows * tile_rows;
    const long r0 = (long)blockIdx.x * per, r1 = min(a.rpw, r0 + per);
    const int ntiles = r1 > r0 ? (int)((r1 - r0 + tile_rows - 1) / tile_rows) : 0;
    uint64_t* full = (uint64_t*)(bns_sm + BNS_RING);
    const uint32_t full0 = bns_smem(full), ring0 = bns_smem(bns_sm);
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * s), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const size_t wbase = (size_t)w * a.rpw * C;           // first element of this worker
    auto issue = [&](int i) {                             // thread 0: fill stage i % stages with tile i
        const int st = i % stages;
        const long row = r0 + (long)(a.reverse ? ntiles - 1 - i : i) * tile_rows;
        const long rows = r1 - row < tile_rows ? r1 - row : tile_rows;
        const uint32_t bytes = (uint32_t)(rows * C * 2), bar = full0 + 8 * st;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes * n_in) : "memory");
        for (int k = 0; k < n_in; ++k)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(ring0 + (st * n_in + k) * BNS_TILE), "l"(a.in[k] + wbase + (size_t)row * C), "r"(bytes), "r"(bar) : "memory");
    };
    if (tid == 0) for (int i = 0; i < stages - 1 && i < ntiles; ++i) issue(i);

    // MODE 3: (sum dy, sum dy xhat) of this worker from the chunk partials of the sums kernel (same grid), while the first
    // tiles are on their way: all threads take part (up to 256 / C interleaved chunk subsets per channel, then a
    // fixed-order sum of the subsets), so every CTA of a worker gets the same sums in the same order.  dgamma / dbeta:
    // CTA i of the launch takes the channels c = i (mod number of CTAs), one warp per channel, lanes over the
    // (worker, chunk) partials and a fixed shuffle tree.
    float2* const red_s = (float2*)(bns_sm + BNS_RING + 64);
    if (MODE == 3) {
        const int chunks = gridDim.x;
        const float2* const part = (const float2*)a.part;
        if (C <= BNV_THREADS) {
            float2* const tmp = red_s + C;                  // [256 / C][C]
            const int nparts = BNV_THREADS / C, c = tid % C, pt = tid / C;
            tmp[pt * C + c] = sum_strided(part + ((size_t)pt * nw + w) * C + c, (size_t)nparts * nw * C, (chunks - pt + nparts - 1) / nparts);
            __syncthreads();
            if (tid < C) {
                float2 t = make_float2(0.f, 0.f);
                for (int q = 0; q < nparts; ++q) { t.x += tmp[q * C + tid].x; t.y += tmp[q * C + tid].y; }
                red_s[tid] = t;
            }
        } else {
            for (int c = tid; c < C; c += BNV_THREADS) red_s[c] = sum_strided(part + (size_t)w * C + c, (size_t)nw * C, chunks);
        }
        {
            const int warp = tid >> 5, lane = tid & 31, rows = nw * chunks, me = w * chunks + blockIdx.x;      // rows = CTAs of the launch
            for (int c = me + warp * rows; c < C; c += (BNV_THREADS / 32) * rows) {
                float2 acc = make_float2(0.f, 0.f);
                for (int r0w = lane; r0w < rows; r0w += 32 * 4) {              // four loads in flight
                    float2 v[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int r = r0w + 32 * j;
                        v[j] = r < rows ? part[((size_t)(r % chunks) * nw + r / chunks) * C + c] : make_float2(0.f, 0.f);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) { acc.x += v[j].x; acc.y += v[j].y; }
                }
                acc = warp_sum2(acc);
                if (lane == 0) { a.dbeta[c] = a.accum_params ? a.dbeta[c] + acc.x : acc.x; a.dgamma[c] = a.accum_params ? a.dgamma[c] + acc.y : acc.y; }
            }
        }
        __syncthreads();
    }
    // Per-channel coefficients, two channels per register pair (the arithmetic below is packed fp32: one instruction per
    // channel pair).  With d = x - mean and scale = gamma * invstd the input gradient gamma * invstd * (dy - c1 - xhat * c2)
    // is scale * dy + (d * ka + kb), ka = -scale * invstd * c2, kb = -scale * c1; sum dy * xhat = invstd * sum dy * d.
    float2 s1[BP], s2[BP], nmean[BP], is[BP], ga[BP], be[BP], sc[BP], ka[BP], kb[BP];
    const float inv_n = 1.f / (float)a.rpw;
#pragma unroll
    for (int j = 0; j < BP; ++j) {
        float* const f1 = &s1[j].x; float* const f2 = &s2[j].x; float* const fnm = &nmean[j].x; float* const fis = &is[j].x;
        float* const fga = &ga[j].x; float* const fbe = &be[j].x; float* const fsc = &sc[j].x; float* const fka = &ka[j].x; float* const fkb = &kb[j].x;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = cg * BV + 2 * j + h;
            const size_t so = ((size_t)w * C + c) * 2;
            f1[h] = 0.f; f2[h] = 0.f;
            if (MODE != 0) { fnm[h] = -a.stats[so]; fis[h] = a.stats[so + 1]; fga[h] = a.gamma[c]; fbe[h] = a.beta[c]; }
            if (MODE == 3) {
                const float c1 = red_s[c].x * inv_n, c2 = red_s[c].y * inv_n;
                fsc[h] = fga[h] * fis[h]; fka[h] = -fsc[h] * fis[h] * c2; fkb[h] = -fsc[h] * c1;
            }
        }
    }
    const bool need_out = (MODE == 1 || MODE == 3) && a.relu && !a.mask_from_x;
    const bool res_in_ring = MODE == 2 && a.res && n_in > 1;
    bool ok = true;
    for (int i = 0; i < ntiles; ++i) {
        // every thread left tile i - 1 at the barrier below, so its stage can take tile i + stages - 1
        if (tid == 0 && i + stages - 1 < ntiles) issue(i + stages - 1);
        const int st = i % stages;
        if (ok && !bns_wait(full0 + 8 * st, (uint32_t)(i / stages) & 1u, a.err)) ok = false;
        const uint8_t* sx = bns_sm + (size_t)(st * n_in) * BNS_TILE + tid * 16;      // row lr, channel group cg: vector lr * cgs + cg = tid + k * 256
        const long trow = r0 + (long)(a.reverse ? ntiles - 1 - i : i) * tile_rows;
        const size_t o0 = wbase + (size_t)trow * C + (size_t)tid * BV;
        const int vec_rows = ok ? (int)min((long)tile_rows, r1 - trow) : 0;            // rows of this tile that exist
        // one 16-byte vector (row rl + k * rows_it of the tile, channel group cg) per call
        auto vec = [&](const int k) {
            const uint4 xw = *(const uint4*)(sx + k * (BNV_THREADS * 16));
            const size_t o = o0 + (size_t)k * (BNV_THREADS * BV);
            float2 xv[BP];
            unpack8(xw, xv);
            if (MODE == 0) {
#pragma unroll
                for (int j = 0; j < BP; ++j) { s1[j] = __fadd2_rn(s1[j], xv[j]); s2[j] = __ffma2_rn(xv[j], xv[j], s2[j]); }
            } else if (MODE == 2) {
#pragma unroll
                for (int j = 0; j < BP; ++j) xv[j] = bn_pair(xv[j], nmean[j], is[j], ga[j], be[j]);
                if (a.res) {
                    float2 rv[BP];
                    unpack8(res_in_ring ? *(const uint4*)(sx + BNS_TILE + k * (BNV_THREADS * 16)) : __ldg((const uint4*)(a.res + o)), rv);
#pragma unroll
                    for (int j = 0; j < BP; ++j) xv[j] = __fadd2_rn(xv[j], rv[j]);
                }
                *(uint4*)(a.y + o) = a.relu ? pack8<true>(xv) : pack8<false>(xv);
            } else {
                float2 dv[BP];
                unpack8(*(const uint4*)(sx + BNS_TILE + k * (BNV_THREADS * 16)), dv);
#pragma unroll
                for (int j = 0; j < BP; ++j) xv[j] = __fadd2_rn(xv[j], nmean[j]);          // d = x - mean from here on
                if (a.relu) {
                    float2 f[BP];
                    if (need_out) unpack8(*(const uint4*)(sx + 2 * BNS_TILE + k * (BNV_THREADS * 16)), f);
                    else {
#pragma unroll
                        for (int j = 0; j < BP; ++j) f[j] = __ffma2_rn(ga[j], __fmul2_rn(xv[j], is[j]), be[j]);   // bn_pair after its first step
                    }
#pragma unroll
                    for (int j = 0; j < BP; ++j) { if (!(f[j].x > 0.f)) dv[j].x = 0.f; if (!(f[j].y > 0.f)) dv[j].y = 0.f; }
                }
                if (MODE == 1) {
#pragma unroll
                    for (int j = 0; j < BP; ++j) { s1[j] = __fadd2_rn(s1[j], dv[j]); s2[j] = __ffma2_rn(dv[j], xv[j], s2[j]); }
                } else {
                    float2 t[BP];
#pragma unroll
                    for (int j = 0; j < BP; ++j) t[j] = __ffma2_rn(sc[j], dv[j], __ffma2_rn(xv[j], ka[j], kb[j]));
                    if (a.accum_dx) {
                        float2 old[BP]; unpack8(*(const uint4*)(a.y + o), old);
#pragma unroll
                        for (int j = 0; j < BP; ++j) t[j] = __fadd2_rn(t[j], old[j]);
                    }
                    *(uint4*)(a.y + o) = pack8<false>(t);
                    if (a.dres) {
                        if (a.accum_dres) {
                            float2 old[BP]; unpack8(*(const uint4*)(a.dres + o), old);
#pragma unroll
                            for (int j = 0; j < BP; ++j) dv[j] = __fadd2_rn(dv[j], old[j]);
                        }
                        *(uint4*)(a.dres + o) = pack8<false>(dv);
                    }
                }
            }
        };
        if (vec_rows == tile_rows) {
            // a whole tile: no per-vector test, so that the four vectors of a thread are independent instruction streams
#pragma unroll
            for (int k = 0; k < BNS_VPT; ++k) vec(k);
        } else {
#pragma unroll
            for (int k = 0; k < BNS_VPT; ++k) if (rl + k * rows_it < vec_rows) vec(k);
        }
        __syncthreads();
    }
    if (MODE == 0 || MODE == 1) {
        // the ring is idle now (every issued tile was waited for): reuse it for the reduction over the row lanes
        float (*red_sh)[2 * BV + 1] = (float (*)[2 * BV + 1])bns_sm;
#pragma unroll
        for (int j = 0; j < BP; ++j) {
            if (MODE == 1) s2[j] = __fmul2_rn(s2[j], is[j]);            // sum dy * d -> sum dy * xhat
            red_sh[tid][2 * j] = s1[j].x; red_sh[tid][2 * j + 1] = s1[j].y; red_sh[tid][BV + 2 * j] = s2[j].x; red_sh[tid][BV + 2 * j + 1] = s2[j].y;
        }
        __syncthreads();
        // thread t < 2*BV*cgs sums one (channel group, value) column over the rows_it row lanes, in a fixed order
        for (int t = tid; t < cgs * 2 * BV; t += BNV_THREADS) {
            const int q = t / (2 * BV), k = t % (2 * BV);
            float acc = 0.f;
            for (int rr = 0; rr < rows_it; ++rr) acc += red_sh[rr * cgs + q][k];
            const int c = q * BV + (k % BV);
            a.part[(((size_t)blockIdx.x * nw + w) * C + c) * 2 + (k / BV)] = acc;
        }
    }
}

// One warp per (worker, channel): lanes take the chunk partials round-robin, then a fixed shuffle tree adds the
// lanes, so the summation order never changes.  stats[w][c] = (mean, invstd).
__global__ void bnv_stats_final(const float* __restrict__ part, float* __restrict__ stats, int chunks, int nwC, long rpw) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (i >= nwC) return;
    float2 a = make_float2(0.f, 0.f);
    for (int k = lane; k < chunks; k += 32) { const float2 v = *(const float2*)(part + ((size_t)k * nwC + i) * 2); a.x += v.x; a.y += v.y; }
    a = warp_sum2(a);
    if (lane == 0) {
        const double mean = (double)a.x / (double)rpw;
        double var = (double)a.y / (double)rpw - mean * mean;
        if (var < 0.0) var = 0.0;
        *(float2*)(stats + (size_t)i * 2) = make_float2((float)mean, (float)(1.0 / sqrt(var + 1e-5)));
    }
}
// same, from the partials a convolution epilogue left: [w * cpw + k][C][2], k < cpw.  One block of 256 threads per
// (worker, 4 channels): a thread owns one channel and every 64th partial, so that a warp's loads cover whole
// 32-byte sectors; then a fixed-order tree over the 64 partial lanes in shared memory.
__global__ void __launch_bounds__(256) bnv_stats_final_tiles(const float* __restrict__ part, float* __restrict__ stats, int cpw, int nw, int C, long rpw) {
    __shared__ float2 sh[64][5];
    const int w = blockIdx.y, tid = threadIdx.x, cl = tid & 3, kl = tid >> 2;
    const int c = blockIdx.x * 4 + cl;
    const float* p = part + ((size_t)w * cpw * C + c) * 2;
    float2 a = make_float2(0.f, 0.f);
    int k = kl;
    for (; k + 448 < cpw; k += 512) {                      // eight independent loads in flight
        float2 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = *(const float2*)(p + (size_t)(k + 64 * j) * C * 2);
        a.x += ((v[0].x + v[1].x) + (v[2].x + v[3].x)) + ((v[4].x + v[5].x) + (v[6].x + v[7].x));
        a.y += ((v[0].y + v[1].y) + (v[2].y + v[3].y)) + ((v[4].y + v[5].y) + (v[6].y + v[7].y));
    }
    for (; k + 192 < cpw; k += 256) {                      // four
        const float2 v0 = *(const float2*)(p + (size_t)k * C * 2), v1 = *(const float2*)(p + (size_t)(k + 64) * C * 2);
        const float2 v2 = *(const float2*)(p + (size_t)(k + 128) * C * 2), v3 = *(const float2*)(p + (size_t)(k + 192) * C * 2);
        a.x += (v0.x + v1.x) + (v2.x + v3.x); a.y += (v0.y + v1.y) + (v2.y + v3.y);
    }
    for (; k < cpw; k += 64) { const float2 v = *(const float2*)(p + (size_t)k * C * 2); a.x += v.x; a.y += v.y; }
    sh[kl][cl] = a;
    __syncthreads();
    for (int d = 32; d > 0; d >>= 1) {
        if (kl < d) { sh[kl][cl].x += sh[kl + d][cl].x; sh[kl][cl].y += sh[kl + d][cl].y; }
        __syncthreads();
    }
    if (kl == 0) {
        const double mean = (double)sh[0][cl].x / (double)rpw;
        double var = (double)sh[0][cl].y / (double)rpw - mean * mean;
        if (var < 0.0) var = 0.0;
        *(float2*)(stats + ((size_t)w * C + c) * 2) = make_float2((float)mean, (float)(1.0 / sqrt(var + 1e-5)));
    }
}
static bool bnv_ok(int dt, int C) { int cgs = C / BV; return dt == 1 && C % BV == 0 && cgs <= BNV_THREADS && (cgs & (cgs - 1)) == 0; }
constexpr int BNS_SMEM = BNS_RING + 8 * 8;
constexpr int BNS_RED_BYTES = BNV_THREADS * BV * 8;   // backward apply: (sum dy, sum dy xhat) per channel, up to 256 * 8 channels (C <= 256: + 256 subset sums)
// Row chunks per worker such that chunks * nw CTAs fill the SMs the caller sizes for once (two CTAs per SM; 0: all SMs),
// each with at least four tiles.
static int bn_device_sms() {
    static int sms = 0;
    if (!sms) { int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); if (sms <= 0) sms = 148; }
    return sms;
}
static int bns_chunks(int nw, long rpw, int C, int sms_wanted) {
    const int sms = sms_wanted > 0 && sms_wanted < bn_device_sms() ? sms_wanted : bn_device_sms();
    const long tile_rows = BNS_TILE / (C * 2);
    long want = ((long)sms * BNS_CTAS) / nw, maxc = (rpw + tile_rows * 4 - 1) / (tile_rows * 4);
    long c = want < maxc ? want : maxc;
    if (c > BNV_MAX_CHUNKS) c = BNV_MAX_CHUNKS;
    return (int)(c < 1 ? 1 : c);
}
template <int MODE>
static void bns_launch(const BnsArgs& a, int chunks, int nw, cudaStream_t s) {
    static bool attr = false;
    constexpr int smem = BNS_SMEM + (MODE == 3 ? BNS_RED_BYTES : 0);
    if (!attr) { cudaFuncSetAttribute(bns_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); attr = true; }
    bns_kernel<MODE><<<dim3(chunks, nw), BNV_THREADS, smem, s>>>(a);
}

bool bn_accepts_conv_partials(int dt, int C) { return bnv_ok(dt, C); }

void bn_forward(int dt, const void* x, const float* gamma, const float* beta, const void* res, void* y, float* stats,
                float* scratch, int nw, long rpw, int C, bool relu, const float* conv_part, int conv_chunks, int sms, int* err, cudaStream_t s) {
    if (bnv_ok(dt, C) && err) {
        const int chunks = bns_chunks(nw, rpw, C, sms);
        const double total = (double)nw * rpw * C;
        BnsArgs a{};
        a.in[0] = (const bf16*)x; a.n_in = 1; a.gamma = gamma; a.beta = beta; a.stats = stats; a.rpw = rpw; a.C = C; a.relu = relu; a.err = err;
        if (conv_part) {
            Scope sc(KC_BN_FWD_STATS, 0.0, 8.0 * conv_chunks * nw * C, s);
            bnv_stats_final_tiles<<<dim3(C / 4, nw), 256, 0, s>>>(conv_part, stats, conv_chunks, nw, C, rpw);
        } else {
            { Scope sc(KC_BN_FWD_STATS, 0.0, 2.0 * total, s);
              BnsArgs r = a; r.part = scratch;
              bns_launch<0>(r, chunks, nw, s); }
            { Scope sc(KC_BN_FWD_STATS, 0.0, 8.0 * chunks * nw * C, s);
              bnv_stats_final<<<cdiv((size_t)nw * C * 32, 256), 256, 0, s>>>(scratch, stats, chunks, nw * C, rpw); }
        }
        Scope sc(KC_BN_FWD_APPLY, 0.0, 2.0 * total * (res ? 3 : 2), s);
        a.y = (bf16*)y; a.res = (const bf16*)res;
        if (res) { a.in[1] = (const bf16*)res; a.n_in = 2; }
        a.reverse = conv_part ? 0 : 1;       // after a statistics pass of its own: x was just read front to back
        bns_launch<2>(a, chunks, nw, s);
        return;
    }
    int chunks = (int)(rpw < RED_CHUNKS ? rpw : RED_CHUNKS);
    dim3 grid(cdiv(C, 32), chunks, nw), blk(32, 8);
    const double esz_ = dt ? 2.0 : 4.0;
    size_t total = (size_t)nw * rpw * C;
    { Scope sc(KC_BN_FWD_STATS, 0.0, esz_ * total, s);
      if (dt) bn_reduce_partial<bf16, false><<<grid, blk, 0, s>>>((const bf16*)x, nullptr, nullptr, nullptr, scratch, rpw, C, false);
      else bn_reduce_partial<float, false><<<grid, blk, 0, s>>>((const float*)x, nullptr, nullptr, nullptr, scratch, rpw, C, false); }
    { Scope sc(KC_BN_FWD_STATS, 0.0, 8.0 * chunks * nw * C, s);
      if (dt) bn_stats_final<bf16><<<cdiv((size_t)nw * C, 128), 128, 0, s>>>(scratch, (const bf16*)x, stats, chunks, nw * C, C, rpw);
      else bn_stats_final<float><<<cdiv((size_t)nw * C, 128), 128, 0, s>>>(scratch, (const float*)x, stats, chunks, nw * C, C, rpw); }
    Scope sc(KC_BN_FWD_APPLY, 0.0, esz_ * total * (res ? 3 : 2), s);
    if (dt) bn_apply_k<bf16><<<cdiv(total, 256), 256, 0, s>>>((const bf16*)x, gamma, beta, (const bf16*)res, (bf16*)y, stats, rpw, C, total, relu);
    else bn_apply_k<float><<<cdiv(total, 256), 256, 0, s>>>((const float*)x, gamma, beta, (const float*)res, (float*)y, stats, rpw, C, total, relu);
}

void bn_backward(int dt, const void* x, const void* out, const void* dout, const float* gamma, const float* beta,
                 const float* stats, void* dx, bool accum_dx, void* dres, bool accum_dres, float* dgamma, float* dbeta, float* red,
                 float* scratch, int nw, long rpw, int C, bool relu, bool has_res, bool accum_params, int sms, int* err, cudaStream_t s) {
    if (bnv_ok(dt, C) && err) {
        const int chunks = bns_chunks(nw, rpw, C, sms);
        const double total = (double)nw * rpw * C;
        const int mask_from_x = relu && !has_res;
        const bool need_out = relu && !mask_from_x;
        const int reads = 2 + (need_out ? 1 : 0);
        BnsArgs a{};
        a.in[0] = (const bf16*)x; a.in[1] = (const bf16*)dout; a.in[2] = (const bf16*)out; a.n_in = reads;
        a.gamma = gamma; a.beta = beta; a.stats = stats; a.rpw = rpw; a.C = C; a.relu = relu; a.mask_from_x = mask_from_x; a.err = err;
        { Scope sc(KC_BN_BWD_REDUCE, 0.0, 2.0 * total * reads, s);
          BnsArgs r = a; r.part = scratch;
          bns_launch<1>(r, chunks, nw, s); }
        Scope sc(KC_BN_BWD_APPLY, 0.0, 2.0 * total * (reads + 1 + (accum_dx ? 1 : 0) + (dres ? (accum_dres ? 2 : 1) : 0)), s);
        a.y = (bf16*)dx; a.accum_dx = accum_dx; a.dres = (bf16*)dres; a.accum_dres = accum_dres;
        a.part = scratch; a.dgamma = dgamma; a.dbeta = dbeta; a.accum_params = accum_params;   // the apply kernel finishes the sums itself
        a.reverse = 1;                       // the sums kernel above has just read the same tensors front to back
        bns_launch<3>(a, chunks, nw, s);
        return;
    }
    int chunks = (int)(rpw < RED_CHUNKS ? rpw : RED_CHUNKS);
    dim3 grid(cdiv(C, 32), chunks, nw), blk(32, 8);
    const double esz_ = dt ? 2.0 : 4.0;
    size_t total = (size_t)nw * rpw * C;
    { Scope sc(KC_BN_BWD_REDUCE, 0.0, esz_ * total * (relu ? 3 : 2), s);
      if (dt) bn_reduce_partial<bf16, true><<<grid, blk, 0, s>>>((const bf16*)x, (const bf16*)out, (const bf16*)dout, stats, scratch, rpw, C, relu);
      else bn_reduce_partial<float, true><<<grid, blk, 0, s>>>((const float*)x, (const float*)out, (const float*)dout, stats, scratch, rpw, C, relu); }
    { Scope sc(KC_BN_BWD_REDUCE, 0.0, 8.0 * chunks * nw * C, s);
      bn_bwd_final<<<cdiv(C, 128), 128, 0, s>>>(scratch, red, dgamma, dbeta, chunks, nw, C, accum_params); }
    Scope sc(KC_BN_BWD_APPLY, 0.0, esz_ * total * ((relu ? 3 : 2) + 1 + (dres ? (accum_dres ? 2 : 1) : 0) + (accum_dx ? 1 : 0)), s);
    if (dt) bn_bwd_apply_k<bf16><<<cdiv(total, 256), 256, 0, s>>>((const bf16*)x, (const bf16*)out, (const bf16*)dout, gamma, stats, red,
                                                                  (bf16*)dx, accum_dx, (bf16*)dres, accum_dres, rpw, C, total, relu);
    else bn_bwd_apply_k<float><<<cdiv(total, 256), 256, 0, s>>>((const float*)x, (const float*)out, (const float*)dout, gamma, stats, red,
                                                                (float*)dx, accum_dx, (float*)dres, accum_dres, rpw, C, total, relu);
}

// ------------------------------------------------------------------------------------------
// softmax cross-entropy: one block; thread i handles rows i, i+256, ...; fixed-order tree sum
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void softmax_ce_k(const float* __restrict__ z, const int32_t* __restrict__ labels, T* __restrict__ dz,
                             float* __restrict__ loss_out, int M, int C, float scale) {
    __shared__ float sh[256];
    float local = 0.f;
    const float inv_m = 1.f / (float)M;
    // exp / log in double: a few thousand values per step, and it keeps the error of (softmax - onehot) at the rounding
    // of the stored result instead of |z| * ulp(expf)
    for (int r = threadIdx.x; r < M; r += blockDim.x) {
        const float* zr = z + (size_t)r * C;
        float m = zr[0];
        for (int c = 1; c < C; ++c) m = fmaxf(m, zr[c]);
        double se = 0.0;
        for (int c = 0; c < C; ++c) se += exp((double)zr[c] - (double)m);
        const double lse = (double)m + log(se);
        int y = labels[r];
        local += (float)(lse - (double)zr[y]);
        for (int c = 0; c < C; ++c) st(dz + (size_t)r * C + c, (float)((exp((double)zr[c] - lse) - (c == y ? 1.0 : 0.0)) * (double)scale));
    }
    sh[threadIdx.x] = local;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) { if ((int)threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s]; __syncthreads(); }
    if (threadIdx.x == 0) *loss_out = sh[0] * inv_m;
}
void softmax_ce(int dt, const float* logits, const int32_t* labels, void* dlogits, float* loss_out, int M, int classes, float scale, cudaStream_t s) {
    Scope sc(KC_SOFTMAX_CE, 0.0, (double)M * classes * (dt ? 6.0 : 8.0) + 4.0 * M, s);
    if (dt) softmax_ce_k<bf16><<<1, 256, 0, s>>>(logits, labels, (bf16*)dlogits, loss_out, M, classes, scale);
    else softmax_ce_k<float><<<1, 256, 0, s>>>(logits, labels, (float*)dlogits, loss_out, M, classes, scale);
}

// ------------------------------------------------------------------------------------------
// Classifier head: the network's last linear layer (c_in -> a few classes) fused with the loss.
//   head_fwd_loss_k : one warp per sample: logits = x W^T + b (fp32, kept for the caller), softmax cross-entropy,
//                     dlogits = (softmax - onehot) * scale in the storage dtype, per-CTA loss partials; the CTA that
//                     finishes last adds the partials in index order (a fixed order) and writes the mean loss.
//   head_bwd_k      : a CTA owns a range of samples: dx = dlogits W (one warp per sample) and the partial sums of
//                     dW[c][k] = sum_rows dlogits[row][c] x[row][k] and db[c] = sum_rows dlogits[row][c] (column k = K).
//   head_reduce_k   : dW / db = partials added in CTA order.
// Replaces an implicit-GEMM launch on 64 x 64 tiles (8-16 CTAs), a one-CTA loss kernel, two bias-gradient launches, a
// split weight gradient with its reduction and an input-gradient launch.  classes <= 16, c_in a multiple of the vector width.
// ------------------------------------------------------------------------------------------
constexpr int HEAD_MAX_C = 16;
constexpr int HEAD_ROWS_PER_CTA = 32;       // samples per CTA of head_bwd_k
template <typename T>
__global__ void __launch_bounds__(256) head_fwd_loss_k(const T* __restrict__ x, const T* __restrict__ W, const float* __restrict__ bias,
                                                       const int32_t* __restrict__ labels, float* __restrict__ logits, T* __restrict__ dz,
                                                       float* __restrict__ loss_part, unsigned* __restrict__ counter, float* __restrict__ loss_out,
                                                       int M, int K, int C, float scale) {
    constexpr int V = Vec<T>::V;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + warp;
    __shared__ float wl[8];
    __shared__ bool last;
    float rloss = 0.f;
    if (row < M) {
        float acc[HEAD_MAX_C];
#pragma unroll
        for (int c = 0; c < HEAD_MAX_C; ++c) acc[c] = 0.f;
        const T* xr = x + (size_t)row * K;
        for (int kv = lane; kv < K / V; kv += 32) {
            float xv[8];
            Vec<T>::load(xr + (size_t)kv * V, xv);
#pragma unroll
            for (int c = 0; c < HEAD_MAX_C; ++c) {
                if (c < C) {
                    float wv[8];
                    Vec<T>::load(W + (size_t)c * K + (size_t)kv * V, wv);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[c] = fmaf(xv[j], wv[j], acc[c]);
                }
            }
        }
        float z = 0.f;                       // lane c keeps logit c
#pragma unroll
        for (int c = 0; c < HEAD_MAX_C; ++c) {
            float v = acc[c];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if (lane == c) z = v + (bias ? bias[c] : 0.f);
        }
        const bool mine = lane < C;
        if (mine) logits[(size_t)row * C + lane] = z;
        float m = mine ? z : -INFINITY;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        // exp / log in double: it keeps the error of (softmax - onehot) at the rounding of the stored result
        double e = mine ? exp((double)z - (double)m) : 0.0;
        double se = e;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) se += __shfl_xor_sync(0xffffffffu, se, d);
        const double lse = (double)m + log(se);
        const int y = labels[row];
        const float zy = __shfl_sync(0xffffffffu, z, y);
        rloss = (float)(lse - (double)zy);
        if (mine) st(dz + (size_t)row * C + lane, (float)((exp((double)z - lse) - (lane == y ? 1.0 : 0.0)) * (double)scale));
    }
    if (lane == 0) wl[warp] = rloss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int i = 0; i < 8; ++i) s += wl[i];
        loss_part[blockIdx.x] = s;
        __threadfence();
        last = atomicAdd(counter, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        float s = 0.f;
        for (unsigned i = 0; i < gridDim.x; ++i) s += ((volatile float*)loss_part)[i];
        *loss_out = s / (float)M;
        *counter = 0u;
    }
}
// grid = ceil(M / HEAD_ROWS_PER_CTA).  part: [CTA][C][K + 1]
template <typename T>
__global__ void __launch_bounds__(256) head_bwd_k(const T* __restrict__ x, const T* __restrict__ W, const T* __restrict__ dz, T* dx, float* __restrict__ part,
                                                  int M, int K, int C, bool accum_dx) {
    constexpr int V = Vec<T>::V;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = blockIdx.x * HEAD_ROWS_PER_CTA, r1 = min(M, r0 + HEAD_ROWS_PER_CTA);
    __shared__ float dzs[HEAD_ROWS_PER_CTA][HEAD_MAX_C];
    for (int i = threadIdx.x; i < (r1 - r0) * C; i += 256) dzs[i / C][i % C] = ld(dz + (size_t)r0 * C + i);
    __syncthreads();
    if (dx) {
        for (int r = r0 + warp; r < r1; r += 8) {
            for (int kv = lane; kv < K / V; kv += 32) {
                float a[8];
#pragma unroll
                for (int j = 0; j < V; ++j) a[j] = 0.f;
                for (int c = 0; c < C; ++c) {
                    float wv[8];
                    Vec<T>::load(W + (size_t)c * K + (size_t)kv * V, wv);
                    const float g = dzs[r - r0][c];
#pragma unroll
                    for (int j = 0; j < V; ++j) a[j] = fmaf(g, wv[j], a[j]);
                }
                T* d = dx + (size_t)r * K + (size_t)kv * V;
                if (accum_dx) {
                    float old[8];
                    Vec<T>::load(d, old);
#pragma unroll
                    for (int j = 0; j < V; ++j) a[j] += old[j];
                }
                Vec<T>::store(d, a);
            }
        }
    }
    // partial sums: (class, vector of V columns) pairs round-robin over the threads, rows in ascending order
    float* out = part + (size_t)blockIdx.x * C * (K + 1);
    const int nkv = K / V;
    for (int p = threadIdx.x; p < C * nkv; p += 256) {
        const int c = p / nkv, kv = p - c * nkv;
        float a[8];
#pragma unroll
        for (int j = 0; j < V; ++j) a[j] = 0.f;
        for (int r = r0; r < r1; ++r) {
            float xv[8];
            Vec<T>::load(x + (size_t)r * K + (size_t)kv * V, xv);
            const float g = dzs[r - r0][c];
#pragma unroll
            for (int j = 0; j < V; ++j) a[j] = fmaf(g, xv[j], a[j]);
        }
#pragma unroll
        for (int j = 0; j < V; ++j) out[(size_t)c * (K + 1) + kv * V + j] = a[j];
    }
    if (threadIdx.x < C) {
        float a = 0.f;
        for (int r = r0; r < r1; ++r) a += dzs[r - r0][threadIdx.x];
        out[(size_t)threadIdx.x * (K + 1) + K] = a;
    }
}
__global__ void head_reduce_k(const float* __restrict__ part, float* __restrict__ dW, float* __restrict__ db, int ctas, int K, int C) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= C * (K + 1)) return;
    float s = 0.f;
    for (int b = 0; b < ctas; ++b) s += part[(size_t)b * C * (K + 1) + i];
    const int c = i / (K + 1), k = i - c * (K + 1);
    if (k < K) dW[(size_t)c * K + k] = s;
    else if (db) db[c] = s;
}
bool head_supported(int dt, int K, int C) { return C >= 2 && C <= HEAD_MAX_C && K % (dt ? 8 : 4) == 0; }
size_t head_scratch_elems(int M, int K, int C) {
    const size_t ctas = (M + HEAD_ROWS_PER_CTA - 1) / HEAD_ROWS_PER_CTA;
    return ctas * C * (K + 1) + (M + 7) / 8;
}
void head_forward_loss(int dt, const void* x, const void* W, const float* bias, const int32_t* labels, float* logits, void* dlogits, float* scratch,
                       unsigned* counter, float* loss_out, int M, int K, int C, float scale, cudaStream_t s) {
    Scope sc(KC_SOFTMAX_CE, 2.0 * M * K * C, (dt ? 2.0 : 4.0) * ((double)M * K + (double)C * K + (double)M * C) + 4.0 * M * C, s);
    const unsigned grid = (M + 7) / 8;
    if (dt) head_fwd_loss_k<bf16><<<grid, 256, 0, s>>>((const bf16*)x, (const bf16*)W, bias, labels, logits, (bf16*)dlogits, scratch, counter, loss_out, M, K, C, scale);
    else head_fwd_loss_k<float><<<grid, 256, 0, s>>>((const float*)x, (const float*)W, bias, labels, logits, (float*)dlogits, scratch, counter, loss_out, M, K, C, scale);
}
void head_backward(int dt, const void* x, const void* W, const void* dlogits, void* dx_or_null, bool accum_dx, float* dW, float* db_or_null, float* scratch,
                   int M, int K, int C, cudaStream_t s) {
    const unsigned ctas = (M + HEAD_ROWS_PER_CTA - 1) / HEAD_ROWS_PER_CTA;
    { Scope sc(KC_FMA_WGRAD, (dx_or_null ? 4.0 : 2.0) * M * K * C, (dt ? 2.0 : 4.0) * ((double)M * K * (dx_or_null ? 2 : 1) + (double)C * K + (double)M * C), s);
      if (dt) head_bwd_k<bf16><<<ctas, 256, 0, s>>>((const bf16*)x, (const bf16*)W, (const bf16*)dlogits, (bf16*)dx_or_null, scratch, M, K, C, accum_dx);
      else head_bwd_k<float><<<ctas, 256, 0, s>>>((const float*)x, (const float*)W, (const float*)dlogits, (float*)dx_or_null, scratch, M, K, C, accum_dx); }
    Scope sc(KC_SPLITK, 0.0, 4.0 * (ctas + 1) * C * (K + 1), s);
    head_reduce_k<<<cdiv((size_t)C * (K + 1), 256), 256, 0, s>>>(scratch, dW, db_or_null, (int)ctas, K, C);
}

// ------------------------------------------------------------------------------------------
// SGD update fused with the emission of the next weight version (Eq. dl_update with P = 11^T/N)
// 128-bit loads and stores; grid sized to a multiple of the SM count by the grid-stride loop.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void sgd_k(float4* __restrict__ master, const float4* __restrict__ grad, T* __restrict__ copy, size_t n4, float lr) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 w = master[i];
        if (grad) {
            float4 g = grad[i];
            w.x = fmaf(-lr, g.x, w.x); w.y = fmaf(-lr, g.y, w.y); w.z = fmaf(-lr, g.z, w.z); w.w = fmaf(-lr, g.w, w.w);
            master[i] = w;
        }
        if (sizeof(T) == 4) {
            ((float4*)copy)[i] = w;
        } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
            uint2 pk; pk.x = *(unsigned*)&lo; pk.y = *(unsigned*)&hi;
            ((uint2*)copy)[i] = pk;
        }
    }
}
void sgd_update(int dt, float* master, const float* grad, void* copy_next, size_t n, float lr, cudaStream_t s) {
    size_t n4 = n / 4;
    if (n4 == 0) return;
    unsigned blocks = cdiv(n4, 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    // per parameter: read master (4) [+ read grad (4) + write master (4)] + write the copy (2 or 4)
    Scope sc(KC_SGD, 0.0, (double)n * ((grad ? 12.0 : 4.0) + (dt ? 2.0 : 4.0)), s);
    if (dt) sgd_k<bf16><<<blocks, 256, 0, s>>>((float4*)master, (const float4*)grad, (bf16*)copy_next, n4, lr);
    else sgd_k<float><<<blocks, 256, 0, s>>>((float4*)master, (const float4*)grad, (float*)copy_next, n4, lr);
}

// ------------------------------------------------------------------------------------------
// General mixing matrix (Eq. dl_update (a), (b)): R replicas of a module's parameters, each with its own gradient.
//   u_r = w_r - lr * g_r ;  w_s(t+1) = sum_r P[s][r] * u_r  (r ascending) ;  copies of w_s(t+1) in the storage dtype.
// A thread owns 4 consecutive parameters of ALL replicas: it reads the R masters (and gradients) first and writes the R
// results afterwards, so the update is in place.  master / grad: [R][n_big + n_small]; the copies of replica r start
// slot_bytes * r after copy0: n_big values in the storage dtype, then n_small floats.
// ------------------------------------------------------------------------------------------
constexpr int MIX_MAX_R = 32;
template <typename T>
__global__ void __launch_bounds__(256) mix_k(float* master, const float* __restrict__ grad, char* copy0, size_t n_big, size_t n_small, size_t slot_bytes,
                                              int R, const float* __restrict__ P, float lr) {
    __shared__ float Ps[MIX_MAX_R * MIX_MAX_R];
    for (int i = threadIdx.x; i < R * R; i += blockDim.x) Ps[i] = P[i];
    __syncthreads();
    const size_t n = n_big + n_small, n4 = n / 4;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 u[MIX_MAX_R];
        for (int r = 0; r < R; ++r) {
            float4 w = ((const float4*)(master + (size_t)r * n))[i];
            if (grad) {
                const float4 g = ((const float4*)(grad + (size_t)r * n))[i];
                w.x = fmaf(-lr, g.x, w.x); w.y = fmaf(-lr, g.y, w.y); w.z = fmaf(-lr, g.z, w.z); w.w = fmaf(-lr, g.w, w.w);
            }
            u[r] = w;
        }
        for (int s = 0; s < R; ++s) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = 0; r < R; ++r) {
                const float p = Ps[s * R + r];
                a.x = fmaf(p, u[r].x, a.x); a.y = fmaf(p, u[r].y, a.y); a.z = fmaf(p, u[r].z, a.z); a.w = fmaf(p, u[r].w, a.w);
            }
            ((float4*)(master + (size_t)s * n))[i] = a;
            char* slot = copy0 + (size_t)s * slot_bytes;
            const size_t e = i * 4;
            if (e < n_big) {
                if (sizeof(T) == 4) ((float4*)slot)[i] = a;
                else {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
                    uint2 pk; pk.x = *(unsigned*)&lo; pk.y = *(unsigned*)&hi;
                    ((uint2*)slot)[i] = pk;
                }
            } else {
                *(float4*)((float*)(slot + n_big * sizeof(T)) + (e - n_big)) = a;
            }
        }
    }
}
int mix_max_replicas() { return MIX_MAX_R; }
void mix_update(int dt, float* master, const float* grad, void* copy0, size_t n_big, size_t n_small, size_t slot_bytes, int R, const float* P, float lr,
                cudaStream_t s) {
    const size_t n4 = (n_big + n_small) / 4;
    if (n4 == 0) return;
    unsigned blocks = cdiv(n4, 256);
    if (blocks > 148 * 4) blocks = 148 * 4;
    Scope sc(KC_SGD, 0.0, (double)R * (n_big + n_small) * ((grad ? 12.0 : 8.0) + (dt ? 2.0 : 4.0)), s);
    if (dt) mix_k<bf16><<<blocks, 256, 0, s>>>(master, grad, (char*)copy0, n_big, n_small, slot_bytes, R, P, lr);
    else mix_k<float><<<blocks, 256, 0, s>>>(master, grad, (char*)copy0, n_big, n_small, slot_bytes, R, P, lr);
}

// ------------------------------------------------------------------------------------------
// schedule tags
// ------------------------------------------------------------------------------------------
__global__ void tags_k(TagOps o) {
    if (threadIdx.x != 0) return;
    // tags of what this step produces first: the last module reads the stash slot it fills itself
    if (o.wr_in) { o.wr_in[0] = o.version_now; o.wr_in[1] = -1; }      // module 1: the batch sampled now
    if (o.wr_out) { o.wr_out[0] = o.fwd_batch; o.wr_out[1] = -1; }
    if (o.wr_stash) { o.wr_stash[0] = o.fwd_batch; o.wr_stash[1] = o.version_now; }
    if (o.wr_grad) { o.wr_grad[0] = o.bwd_batch; o.wr_grad[1] = -1; }
    int64_t fb = o.rd_act ? o.rd_act[0] : -1;
    int64_t bb = -1, bv = -1;
    if (o.rd_stash) {
        bb = o.rd_stash[0];
        if (o.rd_grad && o.rd_grad[0] != bb) bb = -2;
        bv = o.rd_wbwd ? o.rd_wbwd[1] : -1;
        if (o.rd_stash[1] != bv) bv = -2;                 // the stash records the version the forward used
    }
    o.trace[0] = fb; o.trace[1] = bb; o.trace[2] = bv; o.trace[3] = o.rd_wfwd ? o.rd_wfwd[1] : -1;
    // the next weight version replaces a slot only at the end of the step, after the reads above
    if (o.wr_wnext) { o.wr_wnext[0] = -1; o.wr_wnext[1] = o.version_now + 1; }
}
void tags_step(const TagOps& ops, cudaStream_t s) { Scope sc(KC_TAGS, 0.0, 128.0, s); tags_k<<<1, 32, 0, s>>>(ops); }

__global__ void fill_k(float* p, float v, size_t n) { size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; if (i < n) p[i] = v; }
void fill_f32(float* p, float v, size_t n, cudaStream_t s) { if (!n) return; Scope sc(KC_FILL, 0.0, 4.0 * n, s); fill_k<<<cdiv(n, 256), 256, 0, s>>>(p, v, n); }

}  // namespace fdg
