// int8 tensor-core contraction for sm_100a: tcgen05.mma kind::i8 with int32 accumulators in
// tensor memory, operands staged in shared memory by TMA, and the requant / bias / ReLU / int8
// store epilogue fused behind it.  One kernel serves fully connected layers and convolutions.
//
// Convolutions run as "shifted-row" implicit GEMMs.  The activation tensor is stored so that one
// GEMM row is one position (n, Y, X) of a stride-1 grid and every filter tap is a fixed row
// offset: a conv with stride s and window k = s*t on an NHWC tensor is a t x t stride-1 conv on
// its space-to-depth(s) form [H/s][W/s][s*s*C].  The K loop then walks a list of chunks, each a
// TMA box [128 rows][chunk bytes] fetched at (row0 + row_off[j], col_off[j]); rows whose window
// would leave the image are computed and thrown away by the epilogue.
//
// Roles inside a CTA (768 threads): warps 0..3 issue TMA loads, warps 4..7 issue the MMAs (warp 4
// owns the tensor-memory allocation), warps 8..23 are four epilogue warpgroups that drain
// accumulators (each warp its own 32-lane quarter of tensor memory), requantise and store; the
// warpgroups take tiles in turn, or for wide tiles a quarter of the columns each.  The epilogue is
// latency bound per warp, so four warps per scheduler are what keeps the issue slots busy.  The
// kernel is persistent: CTAs stride over the tile list, smem stages and accumulator stages are ring
// buffers guarded by mbarriers.  Every wait is bounded; a wait that gives up sets the policy's
// status word and all roles leave.
//
// Variants, all chosen per launch from TcGemmParams: several output pixels per GEMM row with
// banded weights and a list of 32-byte K steps (kstep_list, px_per_row), rows collected in shared
// memory and stored as whole lines (staged), max-pooling along x on the accumulators (hpool),
// the K loop of a tile split over the issuing warps (ksplit).  The launch is a programmatic
// dependent launch: set-up overlaps the previous launch's tail.
#include <cuda.h>

#include "epilogue.cuh"
#include "internal.h"
#include "tc_gemm.h"
#include "tc_ptx.cuh"

#include <algorithm>
#include <type_traits>

namespace accerl {

namespace {

constexpr int kTileM = 128;
constexpr int kEpiGroups = 4;                       // epilogue warpgroups
constexpr int kMmaWarps = 4;                        // MMA-issuing warps
constexpr int kProdWarps = kMmaWarps;                // TMA-issuing warps, one per MMA warp's ring
constexpr int kThreads = 32 * (kProdWarps + kMmaWarps) + 128 * kEpiGroups;

// Optional per-role stopwatch (build with -DACCERL_TC_TRACE): cycles spent waiting on each barrier
// kind, summed per CTA into the words after the status word.
#ifdef ACCERL_TC_TRACE
#define TRACE_T0() const long long trace_t0_ = clock64()
#define TRACE_ADD(slot) atomicAdd((unsigned long long *)(p.status + 16) + p.trace_slot * 8 + (slot), (unsigned long long)(clock64() - trace_t0_))
#else
#define TRACE_T0()
#define TRACE_ADD(slot)
#endif

struct __align__(8) Barriers {
    uint64_t full[kTcMaxStages], empty[kTcMaxStages];
    uint64_t acc_full[kTcMaxAccStages], acc_empty[kTcMaxAccStages];
    uint64_t b_ready;
    uint64_t raw_full[kProdWarps];   // fused ingest: the raw frame strips of a step have landed
    uint64_t conv_done[kProdWarps];  // fused ingest: the issuing warp has built its tile
    uint32_t tmem_base;
    int abort_flag;
};

// What the epilogue role needs from the kernel's set-up.
struct EpiCtx {
    uint32_t tmem_base, acc_full0, acc_empty0;
    int total_tiles, n_acc, acc_stride, acc_cols, sub;
    int parts, sets_log2;  // K-split: partial accumulators per tile, log2 of the accumulator sets
    const float *s_ks, *s_bs;
    const int *s_skip_mul;
    volatile int *abort_flag;
    uint8_t *staging;  // kStagingBytes per epilogue warp when the layer stores through shared memory
};

enum { kEpiFastDiv = 0, kEpiTieCheck = 1, kEpiLogits = 2, kEpiAffine = 3 };
constexpr int kStagingBytes = 32 * 128;  // 32 rows of 128 output bytes

// byte offset of 16-byte piece `ch` of row `row` in a warp's staging tile; the XOR spreads a
// warp's pieces over the banks both when lanes are rows and when eight lanes share a row
__device__ __forceinline__ int stage_off(int row, int ch) { return row * 128 + ((ch ^ (row & 7)) << 4); }

// 16-byte accesses to a warp's staging tile at 32-bit shared-memory addresses
__device__ __forceinline__ void sts16(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 lds16(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

__device__ __forceinline__ uint4 relu_codes(uint4 v)
{
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int g = 0; g < 4; ++g) w[g] = relu_bytes(w[g]);
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Epilogue role (warps 8..23): drain accumulators, requantise, store.  The per-layer switches are
// template parameters, chosen once per launch, so that the loop over 16-column pieces is straight
// line code: the epilogue is bound by instruction issue.  Rows that are no output position are
// computed like the others and only their stores are skipped, which keeps the warp converged.
//
// STAGED (tiles of 128 columns whose rows are 128 contiguous output bytes): a lane's 16-byte
// pieces would each touch a different 128-byte line of global memory, 32 lines per store
// instruction, and the load/store path then bounds the layer.  Instead every warp collects its 32
// rows in a shared-memory tile and copies it out with eight lanes per row, full lines per
// instruction; the residual source comes in the same way.
template <bool EXTRAS, int MODE, bool RELU, bool PX, bool STAGED, bool KS>
__device__ __forceinline__ void epilogue_role(const TcGemmParams &p, const EpiCtx &c, int warp, int lane)
{
    const uint32_t stage = STAGED ? smem_u32(c.staging + (warp - kProdWarps - kMmaWarps) * kStagingBytes) : 0u;
    const int q = warp & 3;         // this warp's quarter of tensor memory
    const int wg = (warp - kProdWarps - kMmaWarps) >> 2;  // epilogue warpgroup
    const int c_span = p.split_cols ? p.n_tile / kEpiGroups : p.n_tile;
    const int c_begin = p.split_cols ? wg * c_span : 0;
    const int c_end = c_begin + c_span;
    const bool has_skip = EXTRAS && p.skip != nullptr, has_out2 = EXTRAS && p.out2 != nullptr;
    const float s_out = p.s_out, inv_s_out = p.inv_s_out;
    int tile_i = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < c.total_tiles && ok; t += gridDim.x, ++tile_i) {
        if (!p.split_cols && (tile_i % kEpiGroups) != wg) continue;
        int mt = t, nt = 0;
        if (p.n_tiles != 1) {
            mt = t / p.n_tiles;
            nt = t - mt * p.n_tiles;
        }
        // accumulator stage (n_acc is a power of two); with K-split the first of the tile's partials
        const int a = (KS && c.parts > 1) ? (tile_i & ((1 << c.sets_log2) - 1)) * c.parts : tile_i & (c.n_acc - 1);
        const uint32_t apar = (tile_i >> ((KS && c.parts > 1) ? c.sets_log2 : p.n_acc_log2)) & 1;
        {
            TRACE_T0();
            ok = mbar_wait(c.acc_full0 + 8 * a, apar, c.abort_flag, p.status, 16);
            if (threadIdx.x == 32 * (kProdWarps + kMmaWarps)) TRACE_ADD(3);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int col0 = nt * p.n_tile;
        for (int sub = 0; sub < c.sub; ++sub) {
            const int m = (mt * c.sub + sub) * kTileM + q * 32 + lane;
            // which output position is this GEMM row?  Division-free: a float estimate of
            // m / rows_per_image corrected by stepping, a 16.16 reciprocal for the row inside the
            // image (exact for r < 65536), shifts for the power-of-two space-to-depth factor.
            int n = __float2int_rz(__int2float_rn(m) * p.inv_rows_per_image);
            int r = m - n * p.rows_per_image;
            while (r < 0) {
                --n;
                r += p.rows_per_image;
            }
            while (r >= p.rows_per_image) {
                ++n;
                r -= p.rows_per_image;
            }
            const int Y = (int)__umulhi((unsigned)r, p.grid_w_magic), X = r - Y * p.grid_w;
            // PX: the row holds px_per_row output pixels of px_cols columns each
            const int first_px = PX ? X * p.px_per_row : 0;
            const bool valid = n < p.batch && Y < p.out_h && (PX ? first_px < p.px_w : X < p.out_w);
            // columns to store: all, or those of the pixels inside the image
            const int n_store = PX ? min(c_end, (p.px_w - first_px) * p.px_cols) : c_end;
            const int sh = p.out_s2d_log2, smask = (1 << sh) - 1;
            const long long out_row =
                (long long)n * p.out_rows_per_image + (Y >> sh) * p.out_grid_w +
                (PX ? X * p.out_xmul : (X >> sh)) + p.out_row_off;
            int8_t *dst = p.out + out_row * p.out_pitch +
                          ((((Y & smask) << sh) + (X & smask)) * p.n_total) + col0;
            int8_t *dst2 = nullptr;
            const int8_t *skip = nullptr;
            if (EXTRAS) {
                if (has_out2)
                    dst2 = p.out2 + ((long long)n * p.out2_rows_per_image + Y * p.out2_grid_w +
                                     (PX ? X * p.out2_xmul : X) + p.out2_row_off) * p.out2_pitch + col0;
                if (has_skip)
                    skip = p.skip + ((long long)n * p.skip_rows_per_image + Y * p.skip_grid_w +
                                     (PX ? X * p.skip_xmul : X) + p.skip_row_off) * p.skip_pitch + col0;
            }
            float *ldst = MODE == kEpiLogits ? p.logits + (long long)m * p.n_actions : nullptr;
            const uint32_t taddr = c.tmem_base + ((uint32_t)(q * 32) << 16) +
                                   (uint32_t)(a * c.acc_stride + sub * c.acc_cols);
            // staged mode: what the lanes that copy this row in and out need to know about it
            // (offsets in 16-byte units from the tensors' bases; 0 pieces for rows that are no output)
            const int my_pieces = valid ? n_store >> 4 : 0;
            uint32_t my_out16 = 0, my_out2_16 = 0, my_skip16 = 0;
            if (STAGED) {
                my_out16 = (uint32_t)((dst - p.out) >> 4);
                if (has_out2) my_out2_16 = (uint32_t)((dst2 - p.out2) >> 4);
                if (has_skip) {
                    my_skip16 = (uint32_t)((skip - p.skip) >> 4);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = 4 * i + (lane >> 3), ch = lane & 7;
                        const uint32_t so = __shfl_sync(0xffffffffu, my_skip16, r);
                        const int np = __shfl_sync(0xffffffffu, my_pieces, r);
                        uint4 v = make_uint4(0, 0, 0, 0);
                        if (ch < np) v = __ldg(reinterpret_cast<const uint4 *>(p.skip) + so + ch);
                        sts16(stage + (uint32_t)stage_off(r, ch), v);
                    }
                    __syncwarp();
                }
            }
            for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                int acc[16];
                {
                    TRACE_T0();
                    tmem_ld16(taddr + c0, acc);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    for (int part = 1; KS && part < c.parts; ++part) {  // K-split: add the other partial sums
                        int more[16];
                        tmem_ld16(taddr + part * c.acc_stride + c0, more);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int i = 0; i < 16; ++i) acc[i] += more[i];
                    }
                    if (threadIdx.x == 32 * (kProdWarps + kMmaWarps)) TRACE_ADD(7);
                }
                if (c0 + 16 >= c_end && sub == c.sub - 1) {
                    // all of this warp's reads of the stage are done: hand it back to the MMA warp
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(c.acc_empty0 + 8 * a);
                }
                if (EXTRAS && has_skip) {  // residual add in the int32 domain
                    uint4 sv = make_uint4(0, 0, 0, 0);
                    if (STAGED) sv = lds16(stage + (uint32_t)stage_off(lane, c0 >> 4));
                    else if (valid && c0 < n_store) sv = __ldg(reinterpret_cast<const uint4 *>(skip + c0));
                    const uint32_t sw[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        acc[i] += c.s_skip_mul[col0 + c0 + i] * (int)(int8_t)(sw[i >> 2] >> (8 * (i & 3)));
                }
                float ks[16], bs[16];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const float4 kv = *reinterpret_cast<const float4 *>(&c.s_ks[col0 + c0 + 4 * g]);
                    const float4 bv = *reinterpret_cast<const float4 *>(&c.s_bs[col0 + c0 + 4 * g]);
                    ks[4 * g] = kv.x; ks[4 * g + 1] = kv.y; ks[4 * g + 2] = kv.z; ks[4 * g + 3] = kv.w;
                    bs[4 * g] = bv.x; bs[4 * g + 1] = bv.y; bs[4 * g + 2] = bv.z; bs[4 * g + 3] = bv.w;
                }
                if (MODE == kEpiLogits) {
                    if (valid) {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (col0 + c0 + i < p.n_actions)
                                ldst[col0 + c0 + i] = epilogue_float(acc[i], ks[i], bs[i], false);
                    }
                    continue;
                }
                uint32_t w[4];
                if (MODE == kEpiAffine) requant16_affine<RELU>(acc, ks, bs, w);
                else if (MODE == kEpiFastDiv) requant16_fastdiv<RELU>(acc, ks, bs, s_out, inv_s_out, w);
                else requant16(acc, ks, bs, RELU, s_out, inv_s_out, w);
                const uint4 plain = make_uint4(w[0], w[1], w[2], w[3]);
                if (STAGED) {
                    sts16(stage + (uint32_t)stage_off(lane, c0 >> 4), plain);
                } else if (EXTRAS) {
                    uint4 relu = plain;
                    if (p.out_relu | p.out2_relu) {
                        uint32_t wr[4];
#pragma unroll
                        for (int g = 0; g < 4; ++g) wr[g] = relu_bytes(w[g]);
                        relu = make_uint4(wr[0], wr[1], wr[2], wr[3]);
                    }
                    if (valid && c0 < n_store) {
                        *reinterpret_cast<uint4 *>(dst + c0) = p.out_relu ? relu : plain;
                        if (has_out2) *reinterpret_cast<uint4 *>(dst2 + c0) = p.out2_relu ? relu : plain;
                    }
                } else if (valid && c0 < n_store) {
                    *reinterpret_cast<uint4 *>(dst + c0) = plain;
                }
            }
            if (STAGED && MODE != kEpiLogits) {
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = 4 * i + (lane >> 3), ch = lane & 7;
                    const uint32_t o = __shfl_sync(0xffffffffu, my_out16, r);
                    const uint32_t o2 = has_out2 ? __shfl_sync(0xffffffffu, my_out2_16, r) : 0u;
                    const int np = __shfl_sync(0xffffffffu, my_pieces, r);
                    const uint4 v = lds16(stage + (uint32_t)stage_off(r, ch));
                    if (ch < np) {
                        const uint4 vr = (EXTRAS && (p.out_relu | p.out2_relu)) ? relu_codes(v) : v;
                        reinterpret_cast<uint4 *>(p.out)[o + ch] = (EXTRAS && p.out_relu) ? vr : v;
                        if (has_out2) reinterpret_cast<uint4 *>(p.out2)[o2 + ch] = p.out2_relu ? vr : v;
                    }
                }
                __syncwarp();  // the tile is rewritten in the next round
            }
        }
    }
}

// Epilogue for hpool layers (see TcGemmParams::hpool): the warpgroups work in two pairs, each pair
// on every other tile (two tiles are drained at a time, one per accumulator stage); inside a pair a
// warp produces two of the row's four (pooled pixel, 16-channel piece) items, each from the
// accumulators of pixels 2j .. 2j+2.
template <bool RELU, int MODE>
__device__ __forceinline__ void epilogue_hpool(const TcGemmParams &p, const EpiCtx &c, int warp, int lane)
{
    const int q = warp & 3, wg = (warp - kProdWarps - kMmaWarps) >> 2;
    const int pair = wg >> 1, side = wg & 1;
    const float s_out = p.s_out, inv_s_out = p.inv_s_out;
    const int hpc = p.px_cols >> 4;  // 16-channel pieces per pixel: 1 or 2
    int tile_i = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < c.total_tiles && ok; t += gridDim.x, ++tile_i) {
        if ((tile_i & 1) != pair) continue;
        const int a = tile_i & (c.n_acc - 1);
        const uint32_t apar = (tile_i >> p.n_acc_log2) & 1;
        ok = mbar_wait(c.acc_full0 + 8 * a, apar, c.abort_flag, p.status, 16);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int m = t * kTileM + q * 32 + lane;
        int n = __float2int_rz(__int2float_rn(m) * p.inv_rows_per_image);
        int r = m - n * p.rows_per_image;
        while (r < 0) {
            --n;
            r += p.rows_per_image;
        }
        while (r >= p.rows_per_image) {
            ++n;
            r -= p.rows_per_image;
        }
        const int Y = (int)__umulhi((unsigned)r, p.grid_w_magic), X = r - Y * p.grid_w;
        const bool row_ok = n < p.batch && Y < p.out_h;
        int8_t *dst_row = p.out + ((long long)n * p.out_rows_per_image + Y * p.out_grid_w + X * (4 / hpc) +
                                   p.out_row_off) * p.out_pitch;
        const uint32_t tbase = c.tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * c.acc_stride);
#pragma unroll
        for (int item = 0; item < 2; ++item) {
            // 16 channels per pixel: pooled pixels 2 * side + item; 32: pixel `side`, piece `item`
            const int ox = hpc == 1 ? 2 * side + item : side, half = hpc == 1 ? 0 : item;
            const uint32_t taddr = tbase + (uint32_t)(2 * ox * p.px_cols + 16 * half);
            int acc[16], b[16], d[16];
            tmem_ld16(taddr, acc);
            tmem_ld16(taddr + p.px_cols, b);
            tmem_ld16(taddr + 2 * p.px_cols, d);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (item == 1) {  // the last read of the stage: hand it back
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(c.acc_empty0 + 8 * a);
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = max(max(acc[i], b[i]), d[i]);
            float ks[16], bs[16];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const float4 kv = *reinterpret_cast<const float4 *>(&c.s_ks[16 * half + 4 * g]);
                const float4 bv = *reinterpret_cast<const float4 *>(&c.s_bs[16 * half + 4 * g]);
                ks[4 * g] = kv.x; ks[4 * g + 1] = kv.y; ks[4 * g + 2] = kv.z; ks[4 * g + 3] = kv.w;
                bs[4 * g] = bv.x; bs[4 * g + 1] = bv.y; bs[4 * g + 2] = bv.z; bs[4 * g + 3] = bv.w;
            }
            uint32_t w[4];
            if (MODE == kEpiAffine) requant16_affine<RELU>(acc, ks, bs, w);
            else if (MODE == kEpiFastDiv) requant16_fastdiv<RELU>(acc, ks, bs, s_out, inv_s_out, w);
            else requant16(acc, ks, bs, RELU, s_out, inv_s_out, w);
            if (row_ok && X * (4 / hpc) + ox < p.px_w)
                *reinterpret_cast<uint4 *>(dst_row + ox * p.out_pitch + 16 * half) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// Fused input stage: rows [row_begin, row_end) of a step's operand rows (from GEMM row g0 on;
// the tiles of a step are 128 rows apart in one contiguous block) from the raw frame strips
// in shared memory, one lane per row: sixteen 4-byte loads (4 image rows x 4 channel planes), 64
// quantised bytes in (dy, dx, c) order, stored as four 16-byte pieces under the 64-byte swizzle
// (piece index XOR address bits 7..8).  Rows past the last state are zero.  t0 = position of g0
// relative to the first column of the first grid row held in `raw`.
template <int MODE>  // 0: line without the min, 1: line with it, 2: q = u >> 1
__device__ __forceinline__ void convert_tile(const TcGemmParams &p, const uint8_t *raw, uint8_t *tile,
                                             long long g0, int t0, long long total_rows, int row_begin,
                                             int row_end, int lane)
{
    const int Ws = p.grid_w, strip = 4 * p.in_w;
    for (int rr = row_begin + lane; rr < row_end; rr += 32) {
        const unsigned tt = (unsigned)(t0 + rr);
        const int Rrel = (int)__umulhi(tt, p.grid_w_magic), X = (int)tt - Rrel * Ws;
        uint4 q[4] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0),
                      make_uint4(0, 0, 0, 0)};
        if (g0 + rr < total_rows) {
            uint32_t w[4][4];  // [dy][channel]
#pragma unroll
            for (int dy = 0; dy < 4; ++dy)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    w[dy][c] = *reinterpret_cast<const uint32_t *>(raw + (c * p.raw_rows + Rrel) * strip +
                                                                  dy * p.in_w + 4 * X);
#pragma unroll
            for (int dy = 0; dy < 4; ++dy) {
                if (MODE == 2) {
                    q[dy] = ingest_shift_line16(w[dy][0], w[dy][1], w[dy][2], w[dy][3]);
                } else {
                    constexpr bool CL = MODE == 1;
                    q[dy] = make_uint4(
                        ingest_fixed_line4<CL>(w[dy][0], w[dy][1], w[dy][2], w[dy][3], 0, p.ingest_mul, p.ingest_add),
                        ingest_fixed_line4<CL>(w[dy][0], w[dy][1], w[dy][2], w[dy][3], 1, p.ingest_mul, p.ingest_add),
                        ingest_fixed_line4<CL>(w[dy][0], w[dy][1], w[dy][2], w[dy][3], 2, p.ingest_mul, p.ingest_add),
                        ingest_fixed_line4<CL>(w[dy][0], w[dy][1], w[dy][2], w[dy][3], 3, p.ingest_mul, p.ingest_add));
                }
            }
        }
#pragma unroll
        for (int dy = 0; dy < 4; ++dy)
            *reinterpret_cast<uint4 *>(tile + rr * 64 + ((dy ^ ((rr >> 1) & 3)) << 4)) = q[dy];
    }
}

}  // namespace

// EXTRAS compiles in the residual add, the second output and the stored-code ReLU; layers that
// use none of them run the leaner instantiation (the epilogue is bound by instruction issue).
// FUSE is the first conv with the input stage inside (TcGemmParams::fuse_ingest).
// PXK is the kernel for rows of several output pixels; it is kept apart so that its epilogue
// variants do not weigh on the register allocation of the others.
// REQ: the requantiser of the launch's epilogue -- 0: three-step division (or, in the kernels without
// multi-pixel rows, whatever the layer's switches say: logits, tie check), 1: single fma, 2: tie check
// (multi-pixel rows whose output scale failed the division check)
template <bool RESIDENT_B, bool EXTRAS, bool PXK, bool FUSE, int REQ>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const TcGemmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // the dynamic region is only guaranteed 16-byte aligned; swizzled tiles need 1024
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ Barriers bars;
    __shared__ __align__(16) float s_ks[kTcMaxN], s_bs[kTcMaxN];
    __shared__ int s_skip_mul[256];
    if (EXTRAS && p.skip)
        for (int i = threadIdx.x; i < p.n_total && i < 256; i += blockDim.x) s_skip_mul[i] = p.skip_mul[i];
    // per (chunk, k step): low descriptor words of the A and B operands, relative to the stage
    // (B absolute when the weights are resident), so that the issue loop is a load and an add
    __shared__ uint2 s_desc[kTcMaxChunks * 4];
    for (int i = threadIdx.x; i < p.n_total; i += blockDim.x) {
        s_ks[i] = p.kscale[i];
        s_bs[i] = p.bias[i];
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // K-split is only compiled into the kernels with streamed weights (fully connected layers)
    constexpr bool KS = !RESIDENT_B;
    const bool ksplit = KS && p.ksplit;
    const int CH = p.chunk_bytes;
    const int a_chunk_bytes = kTileM * CH;
    const int CHB = p.kstep_list ? 32 : CH;  // bytes of a weight row per chunk
    const int b_tile_bytes = p.n_tile * CHB;
    // shifted mode: a stage is one box of a_rows rows that all taps of the tile read at row offsets
    // sub > 1 (shifted mode only): a pipeline step covers `sub` consecutive 128-row tiles, one TMA
    // box and one accumulator each, so that the barrier round trips are paid once per step
    const int SUB = p.sub;
    // (fused input stage: the tiles of a step overlap in one contiguous block of rows)
    const int box_bytes = FUSE ? kTileM * CH : (p.a_rows * CH + 1023) & ~1023;
    const int stage_bytes = FUSE ? ((((SUB - 1) * kTileM + p.a_rows) * CH + 1023) & ~1023)
                            : p.shifted ? SUB * box_bytes
                                      : p.group * (a_chunk_bytes + (RESIDENT_B ? 0 : b_tile_bytes));
    uint8_t *resident_b = smem;
    uint8_t *stages = smem + (RESIDENT_B ? ((p.n_chunks * b_tile_bytes + 1023) & ~1023) : 0);
    const int n_stages = p.n_stages, n_acc = p.n_acc_stages;
    const int acc_cols = p.n_tile < 32 ? 32 : p.n_tile;  // columns of one accumulator
    const int acc_stride = SUB * acc_cols;               // column stride of an accumulator stage
    volatile int *abort_flag = &bars.abort_flag;

    {
        const int ks_per_chunk = p.kstep_list ? 1 : CH / 32;
        const int Gt = p.shifted ? p.n_chunks : p.group;
        for (int t = threadIdx.x; t < p.n_chunks * ks_per_chunk; t += blockDim.x) {
            const int j = t / ks_per_chunk, k = t - j * ks_per_chunk, cl = j % Gt;
            const uint32_t a_rel = (uint32_t)(p.shifted ? p.row_off[j] * CH + (p.kstep_list ? p.col_off[j] : 0)
                                                        : cl * a_chunk_bytes);
            const uint32_t b_rel =
                RESIDENT_B ? smem_u32(resident_b) + (uint32_t)(j * b_tile_bytes)
                           : (uint32_t)(Gt * a_chunk_bytes + cl * b_tile_bytes);
            s_desc[t] = make_uint2((a_rel >> 4) + 2 * k,
                                   ((b_rel >> 4) + 2 * k) | (RESIDENT_B ? (1u << 16) : 0u));
        }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int a = 0; a < n_acc; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), (!RESIDENT_B && p.ksplit) ? p.n_mma : 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), p.hpool ? 8 : (p.split_cols ? 4 * kEpiGroups : 4));
        }
        mbar_init(smem_u32(&bars.b_ready), 1);
        for (int i = 0; i < kProdWarps; ++i) {
            mbar_init(smem_u32(&bars.raw_full[i]), 1);
            mbar_init(smem_u32(&bars.conv_done[i]), 1);
        }
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kProdWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars.tmem_base)), "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = bars.tmem_base;
    // Programmatic dependent launch: the next tensor-core launch may start its own set-up (barriers,
    // tensor memory, weights) on SMs this grid has left; it waits for this grid's completion before
    // it touches activations (griddepcontrol.wait in the producer and epilogue roles).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int total_tiles = ((p.m_tiles + SUB - 1) / SUB) * p.n_tiles;  // pipeline steps
#ifdef ACCERL_TC_TRACE
    const long long trace_start = clock64();
#endif

    // A smem stage holds `group` consecutive K chunks: [A chunk 0..G-1][B chunk 0..G-1]; the stages
    // of tile i (the CTA's i-th tile) are ring slots i * n_groups .. + n_groups - 1.
    //
    // One thread can only issue a tcgen05.mma every 150..200 cycles, far longer than the tensor
    // pipe needs for the narrow tiles of these layers (measured: two issuing warps double the
    // rate, an N = 64 MMA occupies the pipe for under 50 cycles).  So kMmaWarps warps issue, each
    // for every kMmaWarps-th tile, into their own accumulator stages.
    const int G = p.shifted ? p.n_chunks : p.group, n_groups = p.n_chunks / G;
    const int n_mma = p.n_mma;            // issuing warps in use (never more than accumulators)
    const int ring = n_stages / n_mma;    // ring slots per issuing warp
    const uint32_t stages_addr = smem_u32(stages), resident_addr = smem_u32(resident_b);
    const uint32_t full0 = smem_u32(&bars.full[0]), empty0 = smem_u32(&bars.empty[0]);
    const uint32_t acc_full0 = smem_u32(&bars.acc_full[0]), acc_empty0 = smem_u32(&bars.acc_empty[0]);
    const int my_tiles = blockIdx.x < total_tiles
                             ? (total_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

    if (warp < kProdWarps) {
        // ------------------------------------------------------------- TMA producers (warps 0..3)
        // One wait -> arm -> load round trip takes several hundred cycles and cannot overlap
        // with the next inside one warp, so every issuing warp's ring has a producer of its own.
        const int pw = warp;
        if (pw == 0) {
            if (RESIDENT_B && elect_one()) {
                mbar_expect_tx(smem_u32(&bars.b_ready), (uint32_t)(p.n_chunks * b_tile_bytes));
                for (int j = 0; j < p.n_chunks; ++j)
                    tma_load_2d(resident_addr + j * b_tile_bytes, &map_b, 0, j * p.n_total,
                                smem_u32(&bars.b_ready));
            }
            __syncwarp();
        }
        // the activations are the previous launch's output
        asm volatile("griddepcontrol.wait;" ::: "memory");
        bool ok = true;
        int base_slot = 0;  // ring position of the current tile inside this warp's ring
        uint32_t base_phase = 0;
        int t = blockIdx.x + pw * gridDim.x;
        if constexpr (FUSE) {
            // Fused input stage.  A step's rows are space-to-depth(4) positions (R, X) of uint8 NCHW
            // frames, R = image * grid_h + Y.  The four image rows 4Y .. 4Y+3 of one channel are
            // in_w * 4 contiguous, 16-byte aligned bytes and consecutive Y of an image follow each
            // other, so the raw bytes under a step arrive with at most two bulk copies per channel
            // plane.  This warp then builds the first half of the step's operand rows (the tiles of
            // a step are 128 rows apart in one contiguous block), the ring's issuing warp the second
            // half; both fence their writes to the async proxy.  The ring has one stage and one raw
            // buffer: the next step's strips are fetched
            // as soon as both warps have read the current ones, while the MMAs of this step run.
            const int Ws = p.grid_w, Hs = p.rows_per_image / Ws, strip = 4 * p.in_w;
            const long long total_rows = (long long)p.batch * p.rows_per_image;
            const int raw_bytes = (4 * p.raw_rows * strip + 127) & ~127;
            uint8_t *raw = stages + (size_t)n_stages * stage_bytes + (size_t)pw * raw_bytes;
            const uint32_t raw_bar = smem_u32(&bars.raw_full[pw]);
            const int step_rows = (SUB - 1) * kTileM + p.a_rows;
            auto fetch = [&](int step) {  // elected lane: the raw strips under `step`
                const long long g0 = (long long)step * kTileM * SUB;
                long long g1 = g0 + step_rows;
                if (g1 > total_rows) g1 = total_rows;
                if (g1 <= g0) {
                    mbar_expect_tx(raw_bar, 0);
                    return;
                }
                const int R0 = (int)(g0 / Ws), R1 = (int)((g1 - 1) / Ws);
                mbar_expect_tx(raw_bar, (uint32_t)(4 * (R1 - R0 + 1) * strip));
                const uint32_t dst0 = smem_u32(raw);
                int R = R0;
                while (R <= R1) {  // runs of grid rows inside one image
                    const int n = R / Hs;
                    int Re = (n + 1) * Hs - 1;
                    if (Re > R1) Re = R1;
                    const int Y = R - n * Hs, cnt = Re - R + 1;
                    for (int c = 0; c < 4; ++c)
                        bulk_load(dst0 + (uint32_t)((c * p.raw_rows + (R - R0)) * strip),
                                  p.obs + ((long long)n * 4 + c) * p.in_plane + (long long)Y * strip,
                                  (uint32_t)(cnt * strip), raw_bar);
                    R = Re + 1;
                }
            };
            if (pw < n_mma && pw < my_tiles && elect_one()) fetch(t);
            __syncwarp();
            int k = 0;  // steps done by this warp
            for (int i = pw; i < my_tiles && ok && pw < n_mma; i += n_mma, t += n_mma * gridDim.x, ++k) {
                const int s = pw;  // one stage per ring
                ok = mbar_wait(empty0 + 8 * s, (uint32_t)((k & 1) ^ 1), abort_flag, p.status, 1);
                if (ok) ok = mbar_wait(raw_bar, (uint32_t)(k & 1), abort_flag, p.status, 32);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const long long g0 = (long long)t * kTileM * SUB;
                const int x0 = (int)(g0 % Ws);
                uint8_t *tile = stages + (size_t)s * stage_bytes;
                // this warp converts the first rows of the step, the ring's issuing warp the rest
                const int split = SUB > 1 ? ((step_rows / 2 + 31) & ~31) : step_rows;
                if (p.ingest_clamp == 2) convert_tile<2>(p, raw, tile, g0, x0, total_rows, 0, split, lane);
                else if (p.ingest_clamp) convert_tile<1>(p, raw, tile, g0, x0, total_rows, 0, split, lane);
                else convert_tile<0>(p, raw, tile, g0, x0, total_rows, 0, split, lane);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * s);
                // the issuing warp has read the strips too: fetch the next step's
                ok = mbar_wait(smem_u32(&bars.conv_done[pw]), (uint32_t)(k & 1), abort_flag, p.status, 64);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (i + n_mma < my_tiles && elect_one()) fetch(t + n_mma * gridDim.x);
                __syncwarp();
            }
        }
        // K-split: every warp serves every tile, with the K groups pw, pw + n_mma, ...
        const int tile_step = ksplit ? 1 : n_mma, g_first = ksplit ? pw : 0, g_step = ksplit ? n_mma : 1;
        const int my_groups = g_first < n_groups ? (n_groups - g_first + g_step - 1) / g_step : 0;
        if (ksplit) t = blockIdx.x;
        for (int i = ksplit ? 0 : pw; !FUSE && i < my_tiles && ok && pw < n_mma; i += tile_step, t += tile_step * gridDim.x) {
            int mt = t, nt = 0;
            if (p.n_tiles != 1) {
                mt = t / p.n_tiles;
                nt = t - mt * p.n_tiles;
            }
            const int row0 = mt * kTileM * SUB, brow0 = nt * p.n_tile;
            // Streamed weights: every CTA of a column of tiles reads the same weight chunks, and in
            // lockstep they would all ask the same L2 lines at the same time.  Integer accumulation
            // does not care about the order of K, so each row of tiles starts its K loop at a
            // different group (the stage carries the matching A and B chunks; the issuing side never
            // needs to know which K group a stage holds).
            const int rot = RESIDENT_B ? 0 : mt % n_groups;
            for (int gq = 0; gq < my_groups; ++gq) {
                int gi = g_first + gq * g_step + rot;
                if (gi >= n_groups) gi -= n_groups;
                const int j = gi * G;
                int sl = base_slot + gq;
                uint32_t ph = base_phase;
                while (sl >= ring) {
                    sl -= ring;
                    ph ^= 1;
                }
                const int s = pw + n_mma * sl;
                const uint32_t par = ph ^ 1;
                {
                    TRACE_T0();
                    ok = mbar_wait(empty0 + 8 * s, par, abort_flag, p.status, 1);
                    TRACE_ADD(0);
                }
                if (!ok) break;
                const uint32_t full = full0 + 8 * s;
                const uint32_t st = stages_addr + (uint32_t)s * stage_bytes;
                if (p.shifted) {
                    if (elect_one()) {
                        mbar_expect_tx(full, (uint32_t)(SUB * p.a_rows * CH));
                        for (int sub = 0; sub < SUB; ++sub)
                            tma_load_2d(st + sub * box_bytes, &map_a, 0, row0 + sub * kTileM, full);
                    }
                } else if (elect_one()) {
                    mbar_expect_tx(full, (uint32_t)stage_bytes);
                    for (int c = 0; c < G; ++c) {
                        tma_load_2d(st + c * a_chunk_bytes, &map_a, p.col_off[j + c],
                                    row0 + p.row_off[j + c], full);
                        if (!RESIDENT_B)
                            tma_load_2d(st + G * a_chunk_bytes + c * b_tile_bytes, &map_b, 0,
                                        (j + c) * p.n_total + brow0, full);
                    }
                }
                __syncwarp();
            }
            base_slot += my_groups;
            while (base_slot >= ring) {
                base_slot -= ring;
                base_phase ^= 1;
            }
        }
    } else if (warp < kProdWarps + kMmaWarps) {
        // ------------------------------------------------------------- MMA issuers (warps 4..7)
        const int mw = warp - kProdWarps;
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) |
                               ((uint32_t)(p.n_tile >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
        // descriptor = constant upper word | (address >> 4) in the lower word
        const uint64_t desc_hi =
            (uint64_t)(((uint32_t)(8 * CH) >> 4) | (1u << 14) |
                       ((CH == 128 ? 2u : (CH == 64 ? 4u : 6u)) << 29)) << 32;
        const uint64_t desc_hi_b =
            (uint64_t)(((uint32_t)(8 * CHB) >> 4) | (1u << 14) |
                       ((CHB == 128 ? 2u : (CHB == 64 ? 4u : 6u)) << 29)) << 32;
        const uint32_t desc_lo_flags = 1u << 16;
        const int k_steps = p.kstep_list ? 1 : CH / 32;
        bool ok = true;
        if (RESIDENT_B) ok = mbar_wait(smem_u32(&bars.b_ready), 0, abort_flag, p.status, 2);
        int a = mw, base_slot = 0;
        uint32_t aphase = 0, base_phase = 0;
        const int tile_step = ksplit ? 1 : n_mma, g_first = ksplit ? mw : 0, g_step = ksplit ? n_mma : 1;
        const int my_groups = g_first < n_groups ? (n_groups - g_first + g_step - 1) / g_step : 0;
        for (int i = ksplit ? 0 : mw; i < my_tiles && ok && mw < n_mma; i += tile_step) {
            const uint32_t apar = aphase ^ 1;
            // K-split: the barriers of a tile are those of its first partial accumulator
            const int a_bar = ksplit ? a - mw : a;
            {
                TRACE_T0();
                ok = mbar_wait(acc_empty0 + 8 * a_bar, apar, abort_flag, p.status, 4);
                TRACE_ADD(1);
            }
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t d_tmem = tmem_base + (uint32_t)(a * acc_stride);
            for (int gq = 0; gq < my_groups; ++gq) {
                const int gi = g_first + gq * g_step;
                int sl = base_slot + gq;
                uint32_t par = base_phase;
                while (sl >= ring) {
                    sl -= ring;
                    par ^= 1;
                }
                const int s = mw + n_mma * sl;
                const int j = gi * G;
                if constexpr (FUSE) {
                    // build the step's second operand tile (see the producer role)
                    const int kf = (i - mw) / n_mma;  // steps this warp has done
                    const int raw_bytes = (4 * p.raw_rows * 4 * p.in_w + 127) & ~127;
                    const uint8_t *raw = stages + (size_t)n_stages * stage_bytes + (size_t)mw * raw_bytes;
                    ok = mbar_wait(empty0 + 8 * s, par ^ 1, abort_flag, p.status, 1);
                    if (ok) ok = mbar_wait(smem_u32(&bars.raw_full[mw]), (uint32_t)(kf & 1), abort_flag, p.status, 32);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const int step = (int)blockIdx.x + i * (int)gridDim.x;
                    const long long g0 = (long long)step * kTileM * SUB;
                    const long long total_rows = (long long)p.batch * p.rows_per_image;
                    const int x0 = (int)(g0 % p.grid_w);
                    uint8_t *tile = stages + (size_t)s * stage_bytes;
                    const int step_rows = (SUB - 1) * kTileM + p.a_rows;
                    const int split = SUB > 1 ? ((step_rows / 2 + 31) & ~31) : step_rows;
                    if (p.ingest_clamp == 2) convert_tile<2>(p, raw, tile, g0, x0, total_rows, split, step_rows, lane);
                    else if (p.ingest_clamp) convert_tile<1>(p, raw, tile, g0, x0, total_rows, split, step_rows, lane);
                    else convert_tile<0>(p, raw, tile, g0, x0, total_rows, split, step_rows, lane);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.conv_done[mw]));
                }
                {
                    TRACE_T0();
                    ok = mbar_wait(full0 + 8 * s, par, abort_flag, p.status, 8);
                    TRACE_ADD(2);
                }
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t st_lo = ((stages_addr + (uint32_t)s * stage_bytes) >> 4) | desc_lo_flags;
                if (elect_one()) {
                    const int t0 = j * k_steps, t1 = t0 + G * k_steps;
                    for (int sub = 0; sub < SUB; ++sub) {
                        const uint32_t sub_lo = st_lo + (uint32_t)((sub * box_bytes) >> 4);
                        for (int t = t0; t < t1; ++t) {
                            const uint2 rel = s_desc[t];
                            const uint32_t b_lo = RESIDENT_B ? rel.y : st_lo + rel.y;
                            mma_i8(d_tmem + sub * acc_cols, desc_hi | (sub_lo + rel.x), desc_hi_b | b_lo,
                                   idesc, (uint32_t)(t - g_first * G * k_steps));  // 0: first K step of this warp
                        }
                    }
                    mma_commit(empty0 + 8 * s);  // frees the stage when the MMAs retire
                }
                __syncwarp();
            }
            if (ok && elect_one()) mma_commit(acc_full0 + 8 * a_bar);
            __syncwarp();
            a += n_mma;
            if (a >= n_acc) {
                a -= n_acc;
                aphase ^= 1;
            }
            base_slot += my_groups;
            while (base_slot >= ring) {
                base_slot -= ring;
                base_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------------------- epilogue (warps 8..23)
        EpiCtx c;
        c.tmem_base = tmem_base;
        c.acc_full0 = acc_full0;
        c.acc_empty0 = acc_empty0;
        c.total_tiles = total_tiles;
        c.n_acc = n_acc;
        c.acc_stride = acc_stride;
        c.acc_cols = acc_cols;
        c.sub = SUB;
        c.parts = ksplit ? n_mma : 1;
        c.sets_log2 = 0;
        while ((n_mma << c.sets_log2) < n_acc) ++c.sets_log2;
        c.s_ks = s_ks;
        c.s_bs = s_bs;
        c.s_skip_mul = s_skip_mul;
        c.abort_flag = abort_flag;
        c.staging = stages + (size_t)n_stages * stage_bytes;
        // outputs may reuse buffers that the previous launch still reads
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // (the requantiser is a template parameter of the kernel, not a branch: with both epilogues in
        // one kernel the layers measured slower)
        constexpr bool AFFINE = REQ == 1;
        constexpr int kDivFree = REQ == 1 ? kEpiAffine : (REQ == 2 ? kEpiTieCheck : kEpiFastDiv);
        if constexpr (PXK) {  // multi-pixel rows: one requantiser per kernel
            if (p.hpool) {
                if (p.relu_out) epilogue_hpool<true, kDivFree>(p, c, warp, lane);
                else epilogue_hpool<false, kDivFree>(p, c, warp, lane);
            } else if (p.staged) {
                if (p.relu_out) epilogue_role<EXTRAS, kDivFree, true, true, true, KS>(p, c, warp, lane);
                else epilogue_role<EXTRAS, kDivFree, false, true, true, KS>(p, c, warp, lane);
            } else {
                if (p.relu_out) epilogue_role<EXTRAS, kDivFree, true, true, false, KS>(p, c, warp, lane);
                else epilogue_role<EXTRAS, kDivFree, false, true, false, KS>(p, c, warp, lane);
            }
        } else if constexpr (AFFINE) {
            if (p.relu_out) epilogue_role<EXTRAS, kEpiAffine, true, false, false, KS>(p, c, warp, lane);
            else epilogue_role<EXTRAS, kEpiAffine, false, false, false, KS>(p, c, warp, lane);
        } else {
            if (p.logits_mode) epilogue_role<false, kEpiLogits, false, false, false, KS>(p, c, warp, lane);
            else if (p.fast_div) {
                if (p.relu_out) epilogue_role<EXTRAS, kEpiFastDiv, true, false, false, KS>(p, c, warp, lane);
                else epilogue_role<EXTRAS, kEpiFastDiv, false, false, false, KS>(p, c, warp, lane);
            } else {
                if (p.relu_out) epilogue_role<EXTRAS, kEpiTieCheck, true, false, false, KS>(p, c, warp, lane);
                else epilogue_role<EXTRAS, kEpiTieCheck, false, false, false, KS>(p, c, warp, lane);
            }
        }
    }

#ifdef ACCERL_TC_TRACE
    if (lane == 0 && (warp == 0 || warp == kProdWarps || warp == kProdWarps + kMmaWarps))
        atomicAdd((unsigned long long *)(p.status + 16) + p.trace_slot * 8 + 4 + (warp == 0 ? 0 : (warp == kProdWarps ? 1 : 2)),
                  (unsigned long long)(clock64() - trace_start));
#endif
    // ---------------------------------------------------------------- teardown
    if (*abort_flag) {
        // let copies that are still in flight land before the shared memory goes away
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kProdWarps) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) ==
                cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)sym;
    }
    return fn;
}

// 2-D uint8 tensor [rows][row_bytes] with pitch `pitch`; box [box_rows][box_bytes], swizzled.
accerl_status tc_make_map(void *map_out, const void *base, long long rows, int row_bytes,
                          long long pitch, int box_rows, int box_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) {
        set_error("cuTensorMapEncodeTiled is not available from this driver");
        return ACCERL_ERR_CUDA;
    }
    cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)pitch};
    cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMapSwizzle sw = box_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                            : box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                              : CU_TENSOR_MAP_SWIZZLE_32B;
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void *)base, dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed (%d) for rows=%lld row_bytes=%d pitch=%lld box=%dx%d",
                  (int)r, rows, row_bytes, pitch, box_rows, box_bytes);
        return ACCERL_ERR_CUDA;
    }
    return ACCERL_OK;
}

size_t tc_smem_bytes(const TcGemmParams &p, bool resident_b)
{
    const int a_chunk = kTileM * p.chunk_bytes, b_tile = p.n_tile * (p.kstep_list ? 32 : p.chunk_bytes);
    size_t res = resident_b ? (((size_t)p.n_chunks * b_tile + 1023) & ~(size_t)1023) : 0;
    const size_t stage = p.fuse_ingest
                             ? ((((size_t)(p.sub - 1) * kTileM + p.a_rows) * p.chunk_bytes + 1023) & ~(size_t)1023)
                         : p.shifted ? p.sub * (((size_t)p.a_rows * p.chunk_bytes + 1023) & ~(size_t)1023)
                                   : (size_t)p.group * (a_chunk + (resident_b ? 0 : b_tile));
    const size_t raw = p.fuse_ingest ? (size_t)kProdWarps * ((4 * p.raw_rows * 4 * p.in_w + 127) & ~127) : 0;
    return 1024 + res + (size_t)p.n_stages * stage + (p.staged ? (size_t)4 * kEpiGroups * kStagingBytes : 0) + raw;
}

static int pow2_floor(int v)
{
    int r = 1;
    while (2 * r <= v) r *= 2;
    return r;
}

// Choose ring sizes for a problem; returns false if even the smallest pipeline does not fit.
bool tc_choose_pipeline(TcGemmParams &p, bool resident_b)
{
    const size_t limit = 216 * 1024;  // leaves room for the static shared variables
    // chunks per stage: the largest divisor of n_chunks that keeps a stage at or under 16 KB
    const int per_chunk = kTileM * p.chunk_bytes + (resident_b ? 0 : p.n_tile * p.chunk_bytes);
    p.group = 1;
    for (int g = 1; g <= p.n_chunks; ++g)
        if (p.n_chunks % g == 0 && g * per_chunk <= 16 * 1024) p.group = g;
    const int acc_cols = p.n_tile < 32 ? 32 : p.n_tile;
    // Tiles per pipeline step (shifted mode): as many as still leave two accumulator stages and
    // two shared-memory stages to each issuing warp; otherwise one.
    for (int sub = p.shifted ? p.max_sub : 1; sub >= 1; sub /= 2) {
        p.sub = sub;
        p.n_acc_stages = pow2_floor(std::min(kTcMaxAccStages, 512 / (sub * acc_cols)));
        if (p.n_acc_stages < 1) continue;
        p.n_mma = std::min(kMmaWarps, p.n_acc_stages);
        // wide accumulators leave only two to four stages: give every issuing warp two of them, so
        // that it works on the next tile while the epilogue drains the previous one
        if (sub == 1 && p.shifted && acc_cols >= 128 && p.n_acc_stages >= 2) p.n_mma = p.n_acc_stages / 2;
        const int want = sub > 1 ? 2 * p.n_mma : std::max(2, p.n_mma);
        if (sub > 1 && p.n_acc_stages < 2 * p.n_mma) continue;
        for (int s = kTcMaxStages / p.n_mma * p.n_mma; s >= want; s -= p.n_mma) {
            p.n_stages = s;
            if (tc_smem_bytes(p, resident_b) <= limit) {
                int cols = 32;
                while (cols < p.n_acc_stages * sub * acc_cols) cols *= 2;
                p.tmem_cols = cols;
                p.n_acc_log2 = 0;
                while ((1 << p.n_acc_log2) < p.n_acc_stages) ++p.n_acc_log2;
                // long K loops outside shifted mode: the issuing warps share each tile
                p.ksplit = (!resident_b && !p.shifted && p.n_mma >= 2 && p.n_chunks / p.group >= 2 * p.n_mma) ? 1 : 0;
                return true;
            }
        }
    }
    return false;
}

cudaError_t tc_launch(const void *map_a, const void *map_b, const TcGemmParams &p, bool resident_b,
                      int sm_count, cudaStream_t st)
{
    const size_t smem = tc_smem_bytes(p, resident_b);
    const int tiles = ((p.m_tiles + p.sub - 1) / p.sub) * p.n_tiles;
    const int grid = tiles < sm_count ? tiles : sm_count;
    const bool extras = p.skip || p.out2 || p.out_relu || p.out2_relu;
    // One tile per CTA at most (a fully connected layer at these batch sizes): a single issuing warp
    // then owns every shared-memory stage instead of its share of them, which doubles or
    // quadruples how far the loads run ahead of the MMAs.
    TcGemmParams one = p;
    if (!p.shifted && p.sub == 1 && !p.ksplit && tiles <= sm_count) one.n_mma = 1;
    const TcGemmParams &q = one;
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, *(const CUtensorMap *)map_a, *(const CUtensorMap *)map_b, q);
    };
    cudaError_t e;
    if (p.affine && (!p.fast_div || p.logits_mode)) return cudaErrorInvalidValue;
    auto pick = [&](auto req) -> cudaError_t {
        constexpr int R = decltype(req)::value;
        if constexpr (R == 2) {  // only the multi-pixel kernels have the tie check as a kernel of its own
            if (!p.px_per_row || !resident_b || p.logits_mode) return cudaErrorInvalidValue;
            return extras ? go(tc_gemm_kernel<true, true, true, false, 2>) : go(tc_gemm_kernel<true, false, true, false, 2>);
        } else {
            if (p.px_per_row) {
                if (!resident_b || !p.fast_div || p.logits_mode) return cudaErrorInvalidValue;
                return extras ? go(tc_gemm_kernel<true, true, true, false, R>) : go(tc_gemm_kernel<true, false, true, false, R>);
            }
            if (p.fuse_ingest) {
                if (!resident_b || extras || !p.shifted || p.n_stages != p.n_mma) return cudaErrorInvalidValue;
                return go(tc_gemm_kernel<true, false, false, true, R>);
            }
            return resident_b ? (extras ? go(tc_gemm_kernel<true, true, false, false, R>)
                                        : go(tc_gemm_kernel<true, false, false, false, R>))
                              : (extras ? go(tc_gemm_kernel<false, true, false, false, R>)
                                        : go(tc_gemm_kernel<false, false, false, false, R>));
        }
    };
    e = p.affine ? pick(std::integral_constant<int, 1>())
        : (p.px_per_row && !p.fast_div) ? pick(std::integral_constant<int, 2>()) : pick(std::integral_constant<int, 0>());
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace accerl
