// Parameters of the tensor-core contraction kernel (tc_gemm.cu).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "accerl.h"

namespace accerl {

constexpr int kTcMaxChunks = 64;
constexpr int kTcMaxStages = 12;
constexpr int kTcMaxAccStages = 8;
constexpr int kTcMaxN = 512;

struct TcGemmParams {
    // K loop: chunk j is the TMA box at (row0 + row_off[j], col_off[j]) of the A tensor and rows
    // [j * n_total, (j + 1) * n_total) of the packed weight tensor
    int n_chunks, chunk_bytes;
    int row_off[kTcMaxChunks], col_off[kTcMaxChunks];
    // kstep_list = 1 (shifted mode only): "chunk" j is ONE 32-byte K step, read at byte col_off[j]
    // of row row0 + row_off[j] of the A box; the weights are packed [j][n_total][32 bytes]
    int kstep_list;
    // tiling
    int m_tiles, n_tiles, n_tile, n_total;
    int n_stages, n_acc_stages, n_acc_log2, tmem_cols;
    int group;  // K chunks per shared-memory stage
    int n_mma;  // MMA-issuing warps in use
    // ksplit = 1 (not in shifted mode): the issuing warps share every tile instead of taking tiles in
    // turn -- warp w contracts the K groups w, w + n_mma, ... into an accumulator of its own and the
    // epilogue adds the n_mma partial sums (a K loop of a hundred MMAs is bound by the rate at
    // which one thread can issue them)
    int ksplit;
    // shifted = 1: every chunk reads the same columns at a different row offset, so one TMA box of
    // a_rows = 128 + max(row_off) rows per tile serves all of them (needs resident weights)
    int shifted, a_rows;
    int sub, max_sub;  // 128-row tiles per pipeline step (chosen up to max_sub in shifted mode)
    // GEMM row -> output position: row = n * rows_per_image + Y * grid_w + X, kept when
    // Y < out_h and X < out_w; stored at row n * out_rows_per_image + (Y/s) * out_grid_w + X/s,
    // byte ((Y%s) * s + X%s) * n_total + channel, rows `out_pitch` bytes apart (s = out_s2d)
    int batch, rows_per_image, grid_w, out_h, out_w;
    int out_s2d, out_rows_per_image, out_grid_w, out_pitch;
    int out_s2d_log2;
    int out_row_off;  // added to the output row (a one-pixel border of a padded consumer layout)
    // Several pixels per GEMM row (px_per_row > 0): row (Y, X) holds output pixels
    // X * px_per_row + j, j < px_per_row, px_cols columns each; pixels at or beyond px_w are not
    // stored.  out_xmul scales X in the output row (px_per_row when out_pitch is one pixel).
    int px_per_row, px_cols, px_w;
    int out_xmul, out2_xmul;
    // hpool = 1 (a conv whose only reader is a 3x3 stride-2 max-pool; 16 output channels; the GEMM
    // row holds 9 output pixels, the last one the first of the next row): the epilogue takes the
    // maximum of the ACCUMULATORS of pixels 2j, 2j+1, 2j+2 (j = 0..3) and requantises that -- the
    // requantiser is non-decreasing in the accumulator, so max and requantisation commute -- and
    // stores the 4 horizontally pooled pixels; px_w is then the pooled width, out_xmul = 4.
    int hpool;
    int out_relu;     // clamp the stored codes at 0 (the only reader applies ReLU to its input)
    // optional second copy of the output in another layout: row = n * out2_rows_per_image +
    // Y * out2_grid_w + X + out2_row_off, `out2_pitch` bytes apart, ReLU'd if out2_relu
    int8_t *out2;
    int out2_rows_per_image, out2_grid_w, out2_row_off, out2_pitch, out2_relu;
    // optional residual: acc += skip_mul[c] * skip[row][c], row = n * skip_rows_per_image +
    // Y * skip_grid_w + X * skip_xmul + skip_row_off, rows skip_pitch bytes apart
    const int8_t *skip;
    const int32_t *skip_mul;
    int skip_pitch, skip_rows_per_image, skip_grid_w, skip_xmul, skip_row_off;
    float inv_rows_per_image;  // 1 / rows_per_image, for the division-free row decode
    unsigned grid_w_magic;     // ceil(2^32 / grid_w)
    // epilogue
    const float *kscale, *bias;
    float s_out, inv_s_out;
    int fast_div;  // 1: the three-step division has been verified for this s_out (epilogue.cuh)
    int affine;    // 1: kscale / bias hold the verified single-fma constants (requant_fit.cu)
    int relu_out;
    int split_cols;  // 1: the four epilogue warpgroups share a tile (a quarter of the columns each)
    // 1: rows leave through a shared-memory tile per warp, eight lanes per row (needs n_tile = 128,
    // rows of 128 contiguous output bytes, the verified three-step division, no split_cols)
    int staged;
    int8_t *out;
    int logits_mode;  // 1: write fp32 logits [batch][n_actions] to `logits` instead of int8
    float *logits;
    int n_actions;
    // fuse_ingest = 1 (first conv on 4-channel uint8 frames stored space-to-depth(4), shifted mode,
    // one shared-memory stage per issuing warp): no quantised input tensor exists; the producer
    // warp and the issuing warp of a ring read the raw NCHW frames `obs`, quantise them with
    // q = min((u * ingest_mul + ingest_add) >> 24, 127) and build the operand tiles of a step in
    // shared memory themselves.  in_w = frame width, in_plane = bytes of a channel plane,
    // raw_rows = rows of the input grid a step can touch.
    int fuse_ingest;
    const uint8_t *obs;
    int in_w, in_plane, raw_rows;
    uint32_t ingest_mul, ingest_add;
    int ingest_clamp;  // 0: the line never exceeds 127 for u <= 255, the min is left out; 2: the table is u >> 1
    int *status;
    int trace_slot;  // which block of trace counters a traced build adds to
};

accerl_status tc_make_map(void *map_out, const void *base, long long rows, int row_bytes,
                          long long pitch, int box_rows, int box_bytes);
bool tc_choose_pipeline(TcGemmParams &p, bool resident_b);
size_t tc_smem_bytes(const TcGemmParams &p, bool resident_b);
cudaError_t tc_launch(const void *map_a, const void *map_b, const TcGemmParams &p, bool resident_b,
                      int sm_count, cudaStream_t st);

// uint8 NCHW frames -> int8 space-to-depth(s) rows [B * (H/s) * (W/s)][s*s*C]
cudaError_t launch_ingest_u8_s2d(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int C,
                                 int H, int W, int s, int arith, uint32_t mul, uint32_t add,
                                 cudaStream_t st);
// exhaustive check of the three-step division against the IEEE divide for one output scale
accerl_status verify_fastdiv(float s_out, float inv_s_out, bool relu, float y_max, bool *ok);
accerl_status choose_fastdiv(float s_out, bool relu, float y_max, bool allow, float *inv_s_out, int *fast_div);
accerl_status fit_affine_requant(const float *k, const float *b, int n, float s_out, bool relu,
                                 std::vector<float> *k2, std::vector<float> *b2, bool *ok);
bool fit_ingest_line(const int8_t *lut, uint32_t *mul, uint32_t *add);
bool fit_ingest_float_line(const int8_t *lut, uint32_t mul, uint32_t add, uint32_t *a_bits, uint32_t *c1_bits);

}  // namespace accerl
