// Parameters of the strided-conv kernel on int8 activations (tc_conv.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "accerl.h"

namespace accerl {

struct ConvRowsParams {
    // input: space-to-depth(s) grid of grid_h x grid_w positions per image, row_bytes bytes each;
    // the conv is taps x taps stride 1 on that grid
    int batch, grid_h, grid_w, row_bytes, taps;
    unsigned ws_magic, hs_magic;     // ceil(2^32 / grid_w), ceil(2^32 / grid_h)
    // tiling: a tile is rows_per_tile whole grid rows, a pipeline step tiles_per_step tiles whose
    // operand block arrives as boxes_per_stage TMA boxes of box_rows rows
    int rows_per_tile, max_tiles_per_step, tiles_per_step, total_tiles, total_steps;
    int box_rows, boxes_per_stage, stage_bytes;
    int n_cols;                      // output channels: 16, 32, 48 or 64
    // output: position (n, Y, X) is stored at row n * out_rows_per_image + (Y >> s) * out_grid_w + (X >> s),
    // byte (((Y & m) << s) + (X & m)) * n_total + channel, rows out_pitch bytes apart (s = out_s2d_log2)
    int8_t *out;
    int out_h, out_w, out_s2d_log2, out_rows_per_image, out_grid_w, out_pitch, n_total;
    float s_out, inv_s_out;
    int relu;
    int affine;                      // 1: ks / bs are the single-fma constants (k2, b2)
    alignas(16) float ks[64], bs[64];            // s_in * s_w[c] and bias per output channel
    int *status;
};

bool conv_rows_plan(int grid_h, int grid_w, int row_bytes, int taps, int n_total, long long max_batch,
                    ConvRowsParams *q);
size_t conv_rows_smem_bytes(const ConvRowsParams &q);
cudaError_t conv_rows_launch(const void *map_a, const void *map_b, const ConvRowsParams &q, int batch,
                             int sm_count, cudaStream_t st);

}  // namespace accerl
