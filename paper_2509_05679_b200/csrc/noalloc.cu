// fdg_bias_grad_static: the bias-gradient reduction (column sums of an error-gradient matrix) for
// callers that are not allowed to allocate device memory.  Its scratch lives in a fixed array that is
// part of the library image, so the call itself never touches an allocator.  Self-contained on
// purpose: it shares no kernel with the training step, so nothing in the step's code path changes.
#include "../../include/fdg.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <mutex>
#include <string>

namespace {

constexpr int MAX_CHANNELS = FDG_STATIC_MAX_CHANNELS;    // 4096
constexpr int CHUNKS = 64;                               // row chunks of the first stage
constexpr int MAX_DEVICES = 64;

// [CHUNKS][MAX_CHANNELS] partial sums: 1 MiB per GPU that loads the library, held until the process exits.
static __device__ __align__(256) float g_static_scratch[CHUNKS * MAX_CHANNELS];

// Device address of the array, per device.  In host code `g_static_scratch` is only a handle for the
// runtime; the address a kernel may use comes from cudaGetSymbolAddress with that device current.
float* g_scratch_ptr[MAX_DEVICES] = {};
std::mutex g_mu;
thread_local std::string t_error;

__device__ __forceinline__ float load(const float* p) { return *p; }
__device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// stage 1: block (32 channels x 8 row lanes), grid (channel groups, chunks): part[chunk][c] = sum over the chunk's rows
template <typename T>
__global__ void static_colsum_partial(const T* __restrict__ dy, float* __restrict__ part, long rows, int C, int stride) {
    const int c = blockIdx.x * 32 + threadIdx.x;
    const long per = (rows + gridDim.y - 1) / gridDim.y;
    const long r0 = (long)blockIdx.y * per, r1 = r0 + per < rows ? r0 + per : rows;
    float s = 0.f;
    if (c < C) for (long r = r0 + threadIdx.y; r < r1; r += blockDim.y) s += load(dy + r * C + c);
    __shared__ float sh[8][33];
    sh[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float t = 0.f;
        for (int i = 0; i < 8; ++i) t += sh[i][threadIdx.x];
        part[(size_t)blockIdx.y * stride + c] = t;         // every slot stage 2 reads is written here first
    }
}
// stage 2: out[c] = sum over chunks, ascending (fixed order: repeated calls give identical bits)
__global__ void static_colsum_final(const float* __restrict__ part, float* __restrict__ out, int chunks, int C, int stride) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int i = 0; i < chunks; ++i) s += part[(size_t)i * stride + c];
    out[c] = s;
}

fdg_status fail(fdg_status st, const char* msg) { t_error = msg; return st; }

}  // namespace

extern "C" {

FDG_API const char* fdg_static_last_error(void) { return t_error.c_str(); }

FDG_API fdg_status fdg_bias_grad_static(const void* dev_dy, int32_t dtype, int64_t rows, int32_t channels,
                                        float* dev_db, void* stream) {
    if (!dev_dy || !dev_db) return fail(FDG_ERR_INVALID_ARG, "fdg_bias_grad_static: null pointer");
    if (dtype != 0 && dtype != 1) return fail(FDG_ERR_INVALID_ARG, "fdg_bias_grad_static: dtype must be 0 (fp32) or 1 (bf16)");
    if (rows < 1 || channels < 1) return fail(FDG_ERR_INVALID_ARG, "fdg_bias_grad_static: rows and channels must be positive");
    if (channels > MAX_CHANNELS) {
        char buf[160];
        std::snprintf(buf, sizeof buf, "fdg_bias_grad_static: %d channels exceed the fixed scratch (at most %d)", channels, MAX_CHANNELS);
        return fail(FDG_ERR_INVALID_ARG, buf);
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { cudaGetLastError(); return fail(FDG_ERR_ARCH, "fdg_bias_grad_static: no usable CUDA device"); }
    float* scratch = nullptr;
    {   // one-time set-up per device: ask the runtime where this device keeps the array
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_scratch_ptr[dev]) {
            float* p = nullptr;
            cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                return fail(FDG_ERR_CUDA, (std::string("fdg_bias_grad_static: cudaGetSymbolAddress failed: ") + cudaGetErrorString(e)).c_str());
            }
            g_scratch_ptr[dev] = p;
        }
        scratch = g_scratch_ptr[dev];
    }
    cudaStream_t s = (cudaStream_t)stream;
    const int chunks = (int)(rows < CHUNKS ? rows : CHUNKS);
    dim3 grid((channels + 31) / 32, chunks), blk(32, 8);
    // an error left behind by earlier, unrelated work must not be reported as a failure of these launches
    cudaGetLastError();
    if (dtype) static_colsum_partial<__nv_bfloat16><<<grid, blk, 0, s>>>((const __nv_bfloat16*)dev_dy, scratch, rows, channels, MAX_CHANNELS);
    else static_colsum_partial<float><<<grid, blk, 0, s>>>((const float*)dev_dy, scratch, rows, channels, MAX_CHANNELS);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(FDG_ERR_CUDA, (std::string("fdg_bias_grad_static: launch of the partial sums failed: ") + cudaGetErrorString(e)).c_str());
    static_colsum_final<<<(channels + 127) / 128, 128, 0, s>>>(scratch, dev_db, chunks, channels, MAX_CHANNELS);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(FDG_ERR_CUDA, (std::string("fdg_bias_grad_static: launch of the final sums failed: ") + cudaGetErrorString(e)).c_str());
    return FDG_OK;
}

}  // extern "C"
