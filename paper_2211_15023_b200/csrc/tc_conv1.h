// Parameters of the first-conv kernel with the input stage inside (tc_conv1.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "accerl.h"

namespace accerl {

struct Conv1Params {
    // frames: uint8 [batch][4][in_h][in_w]; grid = space-to-depth(4) positions, grid_h x grid_w per image
    const uint8_t *obs;
    int batch, in_w, in_plane, grid_h, grid_w;
    long long total_grid_rows;       // batch * grid_h
    unsigned ws_magic, hs_magic;     // ceil(2^32 / grid_w), ceil(2^32 / grid_h): division by multiply-high
    // tiling: a tile is rows_per_tile whole grid rows, a pipeline step tiles_per_step tiles
    int rows_per_tile, tiles_per_step, total_tiles, total_steps, stage_bytes;
    int n_cols;                      // output channels: 16 or 32
    // input quantiser: 0 = line q = (u * mul + add) >> 24, 1 = the same with min(., 127), 2 = u >> 1
    int ingest_mode;
    uint32_t ingest_mul, ingest_add;
    // output: position (n, Y, X) is stored at row n * out_rows_per_image + (Y >> s) * out_grid_w + (X >> s),
    // byte (((Y & m) << s) + (X & m)) * n_total + channel, rows out_pitch bytes apart (s = out_s2d_log2)
    int8_t *out;
    int out_h, out_w, out_s2d_log2, out_rows_per_image, out_grid_w, out_pitch, n_total;
    float s_out, inv_s_out;
    int relu;
    int affine;                      // 1: ks / bs are the single-fma constants (k2, b2)
    alignas(16) float ks[32], bs[32];            // s_in * s_w[c] and bias per output channel
    int *status;
};

bool conv1_plan(const accerl_layer_desc &d, int in_h, int in_w, long long max_batch, int n_total,
                int ingest_mode, Conv1Params *q);
size_t conv1_smem_bytes(const Conv1Params &q);
cudaError_t conv1_launch(const void *map_b, const Conv1Params &q, int batch, const uint8_t *obs,
                         int sm_count, cudaStream_t st);

}  // namespace accerl
