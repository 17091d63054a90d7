// First-layer convolution (3x3, stride 1, padding 1, at most 4 input channels, bf16 storage): too thin
// for the tensor cores (K = 27), and bound by writing / reading the 64-channel side once.  Direct
// FMA kernels with register tiles; the weight gradient keeps a 64 x 27 accumulator tile per CTA across
// many pixel tiles and reduces the per-CTA partials in a fixed order.
#include "kernels.h"

#include <cuda_bf16.h>

namespace fdg {

typedef __nv_bfloat16 bf16;
constexpr int ST_THREADS = 256;
constexpr int ST_MAXC = 4;

bool stem_supported(int dt, const ConvGeom& g) {
    auto pow2 = [](int v) { return v > 0 && (v & (v - 1)) == 0; };
    if (dt != 1 || g.C > ST_MAXC || g.R != 3 || g.stride != 1 || g.pad != 1 || g.Co % 64 != 0) return false;
    if (!pow2(g.W) || g.W < 8 || g.W > 64) return false;
    return g.H % (ST_THREADS / g.W) == 0;
}
int stem_wgrad_blocks() { return 4 * 148; }
size_t stem_wgrad_workspace_elems(const ConvGeom& g) { return (size_t)stem_wgrad_blocks() * 64 * 9 * g.C * (g.Co / 64); }

// x tile with a one-pixel zero border, as fp32: xs[(TH+2)][(W+2)][C]
__device__ __forceinline__ void load_x_tile(const bf16* __restrict__ x, float* xs, int n, int h0, int TH, int H, int W, int C) {
    const int tw = W + 2, total = (TH + 2) * tw * C;
    for (int i = threadIdx.x; i < total; i += ST_THREADS) {
        const int ci = i % C; int t = i / C; const int xx = t % tw - 1; const int yy = h0 + t / tw - 1;
        float v = 0.f;
        if (yy >= 0 && yy < H && xx >= 0 && xx < W) v = __bfloat162float(x[(((size_t)n * H + yy) * W + xx) * C + ci]);
        xs[i] = v;
    }
}

// grid (H / TH, N, Co / 64).  thread = (pixel group of 4 along w) x (16 output channels)
__global__ void __launch_bounds__(ST_THREADS) stem_fwd_kernel(const bf16* __restrict__ x, const bf16* __restrict__ w,
                                                              const float* __restrict__ bias, bf16* __restrict__ y,
                                                              int H, int W, int C, int Co, int relu) {
    extern __shared__ float sm[];
    const int TH = ST_THREADS / W, K = 9 * C;
    float* xs = sm;                                   // (TH+2)(W+2)C
    float* ws = sm + (TH + 2) * (W + 2) * C;          // [K][64]
    const int n = blockIdx.y, h0 = blockIdx.x * TH, cob = blockIdx.z * 64;
    load_x_tile(x, xs, n, h0, TH, H, W, C);
    for (int i = threadIdx.x; i < K * 64; i += ST_THREADS) { const int k = i / 64, co = i % 64; ws[i] = __bfloat162float(w[(size_t)(cob + co) * K + k]); }
    __syncthreads();
    const int q = threadIdx.x & 3, pg = threadIdx.x >> 2;
    const int row = pg / (W / 4), col0 = (pg % (W / 4)) * 4;
    float acc[4][16];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[p][j] = 0.f;
    const int tw = W + 2;
    for (int tap = 0; tap < 9; ++tap) {
        const int r = tap / 3, s = tap - r * 3;
        for (int ci = 0; ci < C; ++ci) {
            float xv[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) xv[p] = xs[((row + r) * tw + col0 + p + s) * C + ci];
            const float4* wp = (const float4*)(ws + (tap * C + ci) * 64 + q * 16);
            float wv[16];
#pragma unroll
            for (int j = 0; j < 4; ++j) { const float4 t = wp[j]; wv[4 * j] = t.x; wv[4 * j + 1] = t.y; wv[4 * j + 2] = t.z; wv[4 * j + 3] = t.w; }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[p][j] = fmaf(xv[p], wv[j], acc[p][j]);
        }
    }
    float bv[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) bv[j] = bias ? bias[cob + q * 16 + j] : 0.f;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        uint4 o[2];
        __nv_bfloat162* h = (__nv_bfloat162*)o;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float a = acc[p][2 * j] + bv[2 * j], b = acc[p][2 * j + 1] + bv[2 * j + 1];
            if (relu) { a = fmaxf(a, 0.f); b = fmaxf(b, 0.f); }
            h[j] = __floats2bfloat162_rn(a, b);
        }
        uint4* dst = (uint4*)(y + (((size_t)n * H + h0 + row) * W + col0 + p) * Co + cob + q * 16);
        dst[0] = o[0]; dst[1] = o[1];
    }
}

// grid (blocks, 1, Co / 64): each CTA walks over pixel tiles and keeps dW[64][K] partial sums.
// thread = (4 output channels) x (7 of the K columns) x (one quarter of the tile's pixels)
__global__ void __launch_bounds__(ST_THREADS) stem_wgrad_kernel(const bf16* __restrict__ x, const bf16* __restrict__ dy,
                                                                float* __restrict__ partial, int N, int H, int W, int C, int Co) {
    extern __shared__ float sm[];
    const int TH = ST_THREADS / W, K = 9 * C, tw = W + 2;
    float* xs = sm;                                             // (TH+2)(W+2)C floats
    bf16* dys = (bf16*)(sm + (TH + 2) * tw * C + 4);            // [256][64] bf16 (offset keeps 16-byte alignment below)
    dys = (bf16*)(((uintptr_t)dys + 15) & ~(uintptr_t)15);
    float* red = (float*)(dys + ST_THREADS * 64);               // [64][28]
    const int cob = blockIdx.z * 64;
    const int cg = threadIdx.x & 15, kg = (threadIdx.x >> 4) & 3, ps = threadIdx.x >> 6;
    int off[7]; bool kv[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) {
        const int k = kg * 7 + j; kv[j] = k < K;
        const int kk = kv[j] ? k : 0; const int tap = kk / C, ci = kk - tap * C; const int r = tap / 3, s = tap - r * 3;
        off[j] = (r * tw + s) * C + ci;
    }
    float acc[7][4];
#pragma unroll
    for (int j = 0; j < 7; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
    const int tiles_h = H / TH, tiles = N * tiles_h;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int n = tile / tiles_h, h0 = (tile - n * tiles_h) * TH;
        __syncthreads();                                        // previous tile fully consumed
        load_x_tile(x, xs, n, h0, TH, H, W, C);
        const bf16* src = dy + (((size_t)n * H + h0) * W) * Co + cob;          // 256 pixels x 64 channels (row stride Co)
        for (int i = threadIdx.x; i < ST_THREADS * 8; i += ST_THREADS) {
            const int pix = i >> 3, part = i & 7;
            *(uint4*)(dys + pix * 64 + part * 8) = *(const uint4*)(src + (size_t)pix * Co + part * 8);
        }
        __syncthreads();
#pragma unroll 4
        for (int pi = 0; pi < 64; ++pi) {
            const int pix = ps * 64 + pi;
            const int row = pix / W, col = pix - row * W;
            const uint2 raw = *(const uint2*)(dys + pix * 64 + cg * 4);
            const float2 d01 = __bfloat1622float2(*(const __nv_bfloat162*)&raw.x), d23 = __bfloat1622float2(*(const __nv_bfloat162*)&raw.y);
            const float* xb = xs + (row * tw + col) * C;
            float xv[7];
#pragma unroll
            for (int j = 0; j < 7; ++j) xv[j] = xb[off[j]];          // off[j] of a padded column points at a valid (unused) slot
#pragma unroll
            for (int j = 0; j < 7; ++j) {
                acc[j][0] = fmaf(d01.x, xv[j], acc[j][0]); acc[j][1] = fmaf(d01.y, xv[j], acc[j][1]);
                acc[j][2] = fmaf(d23.x, xv[j], acc[j][2]); acc[j][3] = fmaf(d23.y, xv[j], acc[j][3]);
            }
        }
    }
    // add the four pixel slices in a fixed order, then write this CTA's partial [64][K]
    for (int sl = 0; sl < 4; ++sl) {
        __syncthreads();
        if (ps == sl) {
#pragma unroll
            for (int j = 0; j < 7; ++j)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float* r = red + (cg * 4 + i) * 28 + kg * 7 + j;
                    *r = (sl == 0 ? 0.f : *r) + acc[j][i];
                }
        }
    }
    __syncthreads();
    float* out = partial + ((size_t)blockIdx.z * gridDim.x + blockIdx.x) * 64 * K;
    for (int i = threadIdx.x; i < 64 * K; i += ST_THREADS) { const int co = i / K, k = i - co * K; out[i] = red[co * 28 + k]; }
}

// dw[co][k] = sum over CTAs (ascending) of partial[cz][b][co % 64][k]
__global__ void stem_wgrad_reduce(const float* __restrict__ partial, float* __restrict__ dw, int blocks, int K, int Co, bool accum) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= Co * K) return;
    const int co = i / K, k = i - co * K, cz = co >> 6;
    const float* p = partial + (size_t)cz * blocks * 64 * K + (size_t)(co & 63) * K + k;
    float s = 0.f;
#pragma unroll 8
    for (int b = 0; b < blocks; ++b) s += p[(size_t)b * 64 * K];
    dw[i] = accum ? dw[i] + s : s;
}

void stem_forward(const void* x, const void* w, const float* bias, void* y, const ConvGeom& g, bool relu, cudaStream_t s) {
    const int TH = ST_THREADS / g.W, K = 9 * g.C;
    const size_t smem = ((size_t)(TH + 2) * (g.W + 2) * g.C + (size_t)K * 64) * sizeof(float);
    dim3 grid(g.H / TH, g.N, g.Co / 64);
    const double pix = (double)g.N * g.H * g.W;
    Scope sc(KC_FMA_FWD, 2.0 * pix * g.Co * K, 2.0 * pix * (g.C + g.Co), s);
    stem_fwd_kernel<<<grid, ST_THREADS, smem, s>>>((const bf16*)x, (const bf16*)w, bias, (bf16*)y, g.H, g.W, g.C, g.Co, relu);
}

void stem_wgrad(const void* x, const void* dy, float* dw, float* workspace, const ConvGeom& g, bool accum, cudaStream_t s) {
    const int TH = ST_THREADS / g.W, K = 9 * g.C;
    const size_t smem = ((size_t)(TH + 2) * (g.W + 2) * g.C + 8) * sizeof(float) + 16 + (size_t)ST_THREADS * 64 * 2 + 64 * 28 * sizeof(float);
    static bool attr = false;
    if (!attr) { cudaFuncSetAttribute(stem_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024); attr = true; }
    const int tiles = g.N * (g.H / TH);
    const int blocks = tiles < stem_wgrad_blocks() ? tiles : stem_wgrad_blocks();
    const double pix = (double)g.N * g.H * g.W;
    { Scope sc(KC_FMA_WGRAD, 2.0 * pix * g.Co * K, 2.0 * pix * (g.C + g.Co), s);
      stem_wgrad_kernel<<<dim3(blocks, 1, g.Co / 64), ST_THREADS, smem, s>>>((const bf16*)x, (const bf16*)dy, workspace, g.N, g.H, g.W, g.C, g.Co); }
    Scope sc(KC_SPLITK, 0.0, 4.0 * blocks * g.Co * K, s);
    stem_wgrad_reduce<<<(g.Co * K + 127) / 128, 128, 0, s>>>(workspace, dw, blocks, K, g.Co, accum);
}

}  // namespace fdg
