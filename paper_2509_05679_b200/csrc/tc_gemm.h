// Launch interface of the tcgen05 / TMA kernels (tc_gemm.cu).  bf16 storage only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"

namespace fdg {
namespace tc {

struct alignas(64) TensorMap { unsigned char bytes[128]; };     // a CUtensorMap, opaque here

// Forward / input-gradient kernel.  The "tile domain" is the pixel grid the M tiles enumerate
// (output pixels for forward; for a stride-2 input gradient one parity class of the input pixels).
struct KmParams {
    int Wt, Ht, Nt, tiles_w, tiles_h, tiles_n;   // 128-pixel tile = Wt x Ht x Nt, and how many tiles per axis
    int ntaps, kchunks, xs;                      // filter taps (all classes), 64-channel chunks per tap, coordinate scale of the A map
    int dh[9], dw[9], koff[9];                   // per tap: spatial shift of the A box, column offset into B
    int ncls;                                    // output-parity classes handled by one launch (1, or up to 4 for a stride-2 input gradient)
    int cls_tap0[5];                             // class c uses taps [cls_tap0[c], cls_tap0[c+1])
    int cls_oph[4], cls_opw[4];                  // class c writes domain pixel (h, w) to (h*os + cls_oph[c], w*os + cls_opw[c])
    int N, Hd, Wd;                               // extents of the tile domain (rows outside are not stored)
    int Nfull;                                   // samples in the whole output tensor (N is the end of this launch's group)
    int tma_out;                                 // set by run_km: the epilogue stores through the output tensor map
    int rows_tap[9];                             // set by run_km (rows mode): tap index of (horizontal shift, vertical shift), [dw + 1][dh + 1]
    int n_base;                                  // first sample of the group of workers this launch covers (a multiple of Nt);
                                                 // tiles_n counts the group's tiles, N is the end of the group
    int Ho, Wo, Co, os;                          // output tensor [N,Ho,Wo,Co] and the output stride of a domain pixel
    int Cn;                                      // output channels computed (multiple of the column tile)
    int epi;                                     // EPI_RELU | EPI_ACCUM
    int sms;                                     // SMs the grid is sized for (0: all)
    const float* bias;                           // or nullptr
    void* out;
    float* stat_part;                            // or nullptr: [tile_m * 4 + warp][Cn][2] = (sum, sum of squares) over the
                                                 // warp's 32 output rows, of the values as stored (rounded to bf16)
    int* err;                                    // device word, set non-zero if a bounded wait gave up
};

struct WgParams {
    int Wt, Ht, Nt, tiles_w, tiles_h, tiles_n;   // 64-pixel tile of the dY pixel grid
    int ptiles, ptiles_per_split;
    int n_base;                                  // first sample of the group of workers this launch covers (multiple of Nt)
    int kchunks, row_blocks, xs;                 // 64-channel chunks of c_in; row blocks = taps * kchunks
    int dh[9], dw[9];
    int Co;
    float* partial;                              // [splits][row_blocks * 64][Co]
    int* err;
};

bool init();     // resolves the driver's tensor-map encoder; false if unavailable
// `sms` below (KmParams::sms, the last integer of the other launchers): the SMs a persistent kernel sizes its grid for and
// a weight gradient its contraction splits (0 or >= the device's count: all of them).  Results depend on it only
// through fp32 summation order (split counts).
// NHWC bf16 tensor [N,H,W,C]; box = boxC channels x (boxW x boxH x boxN) pixels; stride 2 samples every other pixel
bool make_map_4d(TensorMap* out, const void* base, int C, int W, int H, int N, int boxC, int boxW, int boxH, int boxN, int stride);
bool make_map_2d(TensorMap* out, const void* base, long inner, long outer, int box_inner, int box_outer);
// Wt x Ht x Nt = pixels, Wt = min(W, pixels) ...; false unless H and W are powers of two
bool pixel_tile(int H, int W, int pixels, int* Wt, int* Ht, int* Nt);

// Output map of run_km: the [N,H,W,C] output tensor with a box of 64 channels x the 32 pixels one epilogue warp owns
// inside a 128-pixel tile of Wt x Ht x Nt pixels.  C must be a multiple of 64.
bool make_map_out(TensorMap* out, const void* base, int C, int W, int H, int N, int Wt, int Ht);

// Tensor maps of one run_km launch.
//   a      : activation, box = 64 channels x one 128-pixel tile (make_map_4d)
//   a_rows : nullptr, or the same tensor with a box of 64 channels x W x (Ht + 2) x 1 pixels: a 3x3 stride-1 layer whose
//            tiles are whole rows of one image then fetches the activation once per horizontal shift ("rows mode")
//   b      : weights, box = 64 x n_tile rows
//   b_half : nullptr, or a map of the same matrix whose box holds n_tile / 2 rows: the kernel then runs as CTA pairs
//            (two SMs share one 256-row MMA and each loads half of B) when the number of pixel tiles is even
//   out    : nullptr, or the output tensor's map from make_map_out: dense outputs are then written by TMA stores
struct KmMaps { const TensorMap* a; const TensorMap* a_rows; const TensorMap* b; const TensorMap* b_half; const TensorMap* out; };
cudaError_t run_km(const KmMaps& m, const KmParams& p, int n_tile, cudaStream_t s);
// accum: dw += the result (second and later groups of workers)
cudaError_t run_wg(const TensorMap& x, const TensorMap& dy, const WgParams& p, int n_tile, int splits, float* dw, bool accum, cudaStream_t s);
// Weight gradient of a 3x3, stride-1, pad-1 layer in rows mode (x is fetched once per horizontal shift and 64-channel
// chunk, dy once per contraction step of 128 pixels).
//   wg_rows_variant: 0 = not supported for this geometry (use run_wg), else the kernel variant
//   wg_rows_splits : CTAs along the contraction for `steps` = 128-pixel steps; the workspace holds that many partial matrices
//   x_rows : x with a box of 64 channels x W x (Ht + 2) x Nt pixels, dy128 : dy with a box of 64 channels x W x Ht x Nt,
//            W x Ht x Nt = 128 pixels
struct WgRowsParams {
    int W, Ht, Nt, tiles_h, tiles_n, n_base;
    int C, Co;
    float* partial;                              // [splits][9 * C][Co]
    int* err;
};
int wg_rows_variant(int H, int W, int C, int Co);
int wg_rows_splits(int variant, int C, int Co, long steps, int sms);
cudaError_t run_wg_rows(const TensorMap& x_rows, const TensorMap& dy128, const WgRowsParams& p, int variant, int splits, float* dw, bool accum,
                        cudaStream_t s);

// Weight gradient of the first layer (3x3, stride 1, pad 1, 3 input channels) on the tensor cores; the im2col lines are
// built in shared memory.  x_raw: x as rows of W * 3 elements with a box of (128 / W + 2) rows (make_map_raw_rows);
// dy128: dy with a box of 64 channels x 128 pixels (make_map_4d).  All N samples; partial: stem_wg_workspace_elems floats.
bool make_map_raw_rows(TensorMap* out, const void* base, int C, int W, int H, int N, int box_rows);
bool stem_wg_supported(int H, int W, int C, int Co);
size_t stem_wg_workspace_elems(int Co, long steps, int sms);
cudaError_t run_stem_wg(const TensorMap& x_raw, const TensorMap& dy128, int H, int W, int N, int Co, float* partial, float* dw, bool accum, int* err,
                        int sms, cudaStream_t s);
// Forward pass of the first layer on the tensor cores (same geometry as run_stem_wg).  out_map: the output's map from
// make_map_out with the tile geometry W x (128 / W) x 1.  w: [Co][27] bf16.  stat_part as in KmParams.
cudaError_t run_stem_fw(const TensorMap& x_raw, const TensorMap& out_map, int H, int W, int N, int Co, const void* w, const float* bias, bool relu,
                        float* stat_part, int* err, int sms, cudaStream_t s);
cudaError_t run_flip_transpose(const void* w, void* wt, int Co, int taps, int Ci, cudaStream_t s);


// The whole update of one module in one launch (see update_module_kernel).
struct UpdOp {                   // weight matrix W[Co][taps][Ci] of a tensor-core layer
    unsigned long long w_off;    // element offset in the module's matrix segment
    int Co, taps, Ci;
    int tile0;                   // first 32 x 32 tile of this matrix in the launch
};
struct UpdRange { unsigned long long start, count; };   // elements (multiples of 4) outside those matrices
struct UpdTable {
    int nops, nranges, total_tiles;
    unsigned long long n_big;    // elements of the matrix segment; the vector segment follows it
    UpdOp ops[12];
    UpdRange ranges[14];
};
cudaError_t run_update_module(const UpdTable& tb, float* master, const float* grad, void* wcopy, void* wtcopy, float* small_copy, float lr,
                              bool has_grad, cudaStream_t s);
}  // namespace tc
}  // namespace fdg
