// Strided, unpadded convolutions on int8 activations (the second and third layer of the paper's
// Atari networks, table "network architecture and inference time") in the form the first-conv
// kernel has: a conv with stride s and window k = s * t on a tensor stored space-to-depth(s) is a
// t x t stride-1 conv on its grid, one GEMM row per grid position, every tap a fixed row offset of
// ONE operand block in shared memory.
//
// What differs from the general contraction kernel (tc_gemm.cu):
// - a tile is S whole grid rows (S * Ws <= 128 GEMM rows): a thread of the epilogue owns the same
//   (row, X) of every tile, its output address costs two multiplies per tile;
// - a pipeline step is T tiles whose operand block (the T * S grid rows and the t - 1 rows the taps
//   reach into) arrives by a few TMA boxes issued by one warp; kStages2 blocks are in flight;
// - four warps issue the MMAs, tiles in turn (descriptors computed in registers; one warp that
//   shares its scheduler with five others issues an instruction every six to eight cycles, and a
//   tile takes some two hundred: measured 49 / 41 / 36 us for the layer with one / two / four
//   issuing warps), sixteen warps drain accumulators; scales and biases are kernel parameters read from the constant bank, because
//   shared-memory loads of the epilogue queue behind the operand reads of the MMAs.
//
// Every wait is bounded; a wait that gives up sets the status word and all roles leave.
#include <cuda.h>

#include <algorithm>

#include "epilogue.cuh"
#include "internal.h"
#include "tc_conv.h"
#include "tc_ptx.cuh"

namespace accerl {

namespace {

constexpr int kMmaWarps2 = 4;            // warps 0..3 issue MMAs, the CTA's tiles in turn
constexpr int kEpiWarps2 = 16;           // warps 4..19 drain accumulators
constexpr int kWarps2 = 4 + kEpiWarps2 + 1;  // the last warp issues the TMA loads
constexpr int kThreads2 = 32 * kWarps2;
constexpr int kStages2 = 4;
constexpr int kMaxSlots2 = 16;

struct __align__(8) Bars2 {
    uint64_t full[kStages2], empty[kStages2];
    uint64_t acc_full[kMaxSlots2], acc_empty[kMaxSlots2];
    uint64_t b_ready;
    uint32_t tmem_base;
    int abort_flag;
};

}  // namespace

// TAPS_T / RB_T: taps per side and bytes of an operand row as compile-time constants (0 = taken from
// the parameters); with them the issue loop of a tile is straight-line code, and the issuing warps'
// instruction count is what bounds how fast tiles start.
template <int NCOLS, int TAPS_T, int RB_T, bool AFFINE>
__global__ void __launch_bounds__(kThreads2, 1)
conv_rows_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ ConvRowsParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw2[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw2 + 1023) & ~(uintptr_t)1023);
    __shared__ Bars2 bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kSlotCols = NCOLS <= 32 ? 32 : 64;     // tensor-memory columns of one accumulator
    constexpr int kAccSlots = 512 / kSlotCols;
    const int RB = RB_T ? RB_T : p.row_bytes, taps = TAPS_T ? TAPS_T : p.taps, n_taps = taps * taps;
    const int b_bytes = n_taps * NCOLS * RB;
    uint8_t *b_tiles = smem;
    uint8_t *stages = smem + ((b_bytes + 1023) & ~1023);
    const int stage_bytes = p.stage_bytes;
    volatile int *abort_flag = &bars.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages2; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), kMmaWarps2);
        }
        for (int a = 0; a < kAccSlots; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);
        }
        mbar_init(smem_u32(&bars.b_ready), 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&bars.tmem_base)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = bars.tmem_base;
    // the next launch may set itself up while this grid drains
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int T = p.tiles_per_step, S = p.rows_per_tile, Ws = p.grid_w, Hs = p.grid_h;
    const int my_steps = (int)blockIdx.x < p.total_steps
                             ? (p.total_steps - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const uint32_t full0 = smem_u32(&bars.full[0]), empty0 = smem_u32(&bars.empty[0]);
    const uint32_t acc_full0 = smem_u32(&bars.acc_full[0]), acc_empty0 = smem_u32(&bars.acc_empty[0]);

    if (warp < kMmaWarps2) {
        // ------------------------------------------------------------------ MMA issuers
        if (warp == 0 && elect_one()) {
            mbar_expect_tx(smem_u32(&bars.b_ready), (uint32_t)b_bytes);
            for (int j = 0; j < n_taps; ++j)
                tma_load_2d(smem_u32(b_tiles) + j * NCOLS * RB, &map_b, 0, j * NCOLS, smem_u32(&bars.b_ready));
        }
        __syncwarp();
        bool ok = mbar_wait(smem_u32(&bars.b_ready), 0, abort_flag, p.status, 2);
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NCOLS >> 3) << 17) |
                               ((uint32_t)(128 >> 4) << 24);
        // swizzled K-major rows of RB bytes: descriptor = constant upper word | (address >> 4)
        const uint64_t desc_hi =
            (uint64_t)(((uint32_t)(8 * RB) >> 4) | (1u << 14) | ((RB == 128 ? 2u : (RB == 64 ? 4u : 6u)) << 29)) << 32;
        const uint32_t lo_flags = 1u << 16;
        const uint32_t b_lo = (smem_u32(b_tiles) >> 4) | lo_flags;
        const uint32_t row16 = (uint32_t)(RB >> 4), ksteps = (uint32_t)(RB >> 5);
        const uint32_t b_tap = (uint32_t)(NCOLS * RB) >> 4;
        for (int k = 0; k < my_steps && ok; ++k) {
            const int step = (int)blockIdx.x + k * (int)gridDim.x;
            const int s = k % kStages2;
            ok = mbar_wait(full0 + 8 * s, (uint32_t)((k / kStages2) & 1), abort_flag, p.status, 8);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t st_lo = ((smem_u32(stages) + (uint32_t)(s * stage_bytes)) >> 4) | lo_flags;
            for (int i = 0; i < T && ok; ++i) {
                if (step * T + i >= p.total_tiles) break;
                const int seq = k * T + i, slot = seq % kAccSlots;  // the CTA's tiles in order
                if (seq % kMmaWarps2 != warp) continue;
                ok = mbar_wait(acc_empty0 + 8 * slot, (uint32_t)(((seq / kAccSlots) & 1) ^ 1), abort_flag, p.status, 4);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (elect_one()) {
                    const uint32_t d = tmem_base + (uint32_t)(slot * kSlotCols);
                    const uint32_t a_tile = st_lo + (uint32_t)(i * S * Ws) * row16;
                    if constexpr (TAPS_T != 0 && RB_T != 0) {
                        const uint32_t a_row = (uint32_t)Ws * row16;
#pragma unroll
                        for (int ty = 0; ty < TAPS_T; ++ty)
#pragma unroll
                            for (int tx = 0; tx < TAPS_T; ++tx)
#pragma unroll
                                for (int ks = 0; ks < RB_T / 32; ++ks)
                                    mma_i8(d, desc_hi | (a_tile + ty * a_row + (uint32_t)(tx * (RB_T / 16) + 2 * ks)),
                                           desc_hi | (b_lo + (uint32_t)((ty * TAPS_T + tx) * (NCOLS * RB_T / 16) + 2 * ks)),
                                           idesc, (uint32_t)(ty | tx | ks));
                    } else {
                        uint32_t b_j = b_lo, first = 0;
                        for (int ty = 0; ty < taps; ++ty) {
                            uint32_t a_j = a_tile + (uint32_t)(ty * Ws) * row16;
                            for (int tx = 0; tx < taps; ++tx) {
                                for (uint32_t ks = 0; ks < ksteps; ++ks) {
                                    mma_i8(d, desc_hi | (a_j + 2 * ks), desc_hi | (b_j + 2 * ks), idesc, first);
                                    first = 1;
                                }
                                a_j += row16;
                                b_j += b_tap;
                            }
                        }
                    }
                    mma_commit(acc_full0 + 8 * slot);
                }
                __syncwarp();
            }
            if (ok && elect_one()) mma_commit(empty0 + 8 * s);  // the block is free when these MMAs retire
            __syncwarp();
        }
    } else if (warp == kWarps2 - 1) {
        // ------------------------------------------------------------------ TMA producer
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the activations are the previous launch's output
        bool ok = true;
        for (int k = 0; k < my_steps && ok; ++k) {
            const int step = (int)blockIdx.x + k * (int)gridDim.x;
            const int s = k % kStages2;
            ok = mbar_wait(empty0 + 8 * s, (uint32_t)(((k / kStages2) & 1) ^ 1), abort_flag, p.status, 1);
            if (!ok) break;
            if (elect_one()) {
                const uint32_t full = full0 + 8 * s;
                const uint32_t dst = smem_u32(stages) + (uint32_t)(s * stage_bytes);
                const int row0 = step * T * S * Ws;  // first grid position of the step
                mbar_expect_tx(full, (uint32_t)(p.boxes_per_stage * p.box_rows * RB));
                for (int b = 0; b < p.boxes_per_stage; ++b)
                    tma_load_2d(dst + (uint32_t)(b * p.box_rows * RB), &map_a, 0, row0 + b * p.box_rows, full);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - 4, wg = ew >> 2, q = warp & 3;
        constexpr int kGroups = kEpiWarps2 / 4;
        const int r = q * 32 + lane;  // this thread's row of every tile
        const int Rl = (int)__umulhi((unsigned)r, p.ws_magic), X = r - Rl * Ws;
        const int sh = p.out_s2d_log2, smask = (1 << sh) - 1;
        const bool row_ok = r < S * Ws && X < p.out_w;
        const int x_off = (X >> sh) * p.out_pitch + (X & smask) * p.n_total;
        const float s_out = p.s_out, inv_s_out = p.inv_s_out;
        asm volatile("griddepcontrol.wait;" ::: "memory");  // the output may reuse a buffer an earlier launch reads
        bool ok = true;
        // warpgroup wg takes the CTA's tiles wg, wg + kGroups, ... (seq: the CTA's tiles in order;
        // T is 1, 2 or 4)
        const int t_log2 = T == 4 ? 2 : (T == 2 ? 1 : 0);
        for (int seq = wg; ok; seq += kGroups) {
            {
                const int k = seq >> t_log2, i = seq & (T - 1);
                if (k >= my_steps) break;
                const int tile = ((int)blockIdx.x + k * (int)gridDim.x) * T + i;
                if (tile >= p.total_tiles) break;  // only the last step is short, and later tiles lie behind it
                const int slot = seq % kAccSlots;
                ok = mbar_wait(acc_full0 + 8 * slot, (uint32_t)((seq / kAccSlots) & 1), abort_flag, p.status, 16);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(slot * kSlotCols);
                const unsigned R = (unsigned)(tile * S + Rl);
                const unsigned n = __umulhi(R, p.hs_magic);
                const int Y = (int)(R - n * (unsigned)Hs);
                const bool valid = row_ok && Y < p.out_h && (int)n < p.batch;
                int8_t *dst = p.out + (size_t)(n * (unsigned)p.out_rows_per_image + (unsigned)((Y >> sh) * p.out_grid_w)) *
                                          (size_t)p.out_pitch +
                              (((Y & smask) << sh) * p.n_total + x_off);
                constexpr int kHalves = (NCOLS + 31) / 32;  // 32 columns at a time
#pragma unroll
                for (int hh = 0; hh < kHalves; ++hh) {
                    constexpr int kPieces = NCOLS >= 32 ? 2 : 1;
                    int acc[kPieces][16];
#pragma unroll
                    for (int h = 0; h < kPieces; ++h) tmem_ld16(taddr + 32 * hh + 16 * h, acc[h]);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    if (hh == kHalves - 1) {  // the last read of the accumulator: hand it back
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_empty0 + 8 * slot);
                    }
                    uint32_t wq[kPieces][4];
#pragma unroll
                    for (int h = 0; h < kPieces; ++h) {
                        if (32 * hh + 16 * h >= NCOLS) continue;
                        float ks[16], bs[16];
#pragma unroll
                        for (int g = 0; g < 4; ++g) {  // kernel parameters: 16-byte reads from the constant bank
                            const float4 kv = *reinterpret_cast<const float4 *>(&p.ks[32 * hh + 16 * h + 4 * g]);
                            const float4 bv = *reinterpret_cast<const float4 *>(&p.bs[32 * hh + 16 * h + 4 * g]);
                            ks[4 * g] = kv.x; ks[4 * g + 1] = kv.y; ks[4 * g + 2] = kv.z; ks[4 * g + 3] = kv.w;
                            bs[4 * g] = bv.x; bs[4 * g + 1] = bv.y; bs[4 * g + 2] = bv.z; bs[4 * g + 3] = bv.w;
                        }
                        uint32_t (&wv)[4] = wq[h];
                        if (AFFINE) {
                            if (p.relu) requant16_affine<true>(acc[h], ks, bs, wv);
                            else requant16_affine<false>(acc[h], ks, bs, wv);
                        } else {
                            if (p.relu) requant16_fastdiv<true>(acc[h], ks, bs, s_out, inv_s_out, wv);
                            else requant16_fastdiv<false>(acc[h], ks, bs, s_out, inv_s_out, wv);
                        }
                    }
                    if (valid) {  // 32 channels in one store where the channel count is a multiple of 32
                        if constexpr (NCOLS % 32 == 0) {  // positions are then 32-byte aligned
                            stg32(dst + 32 * hh, wq[0], wq[1]);
                        } else {
#pragma unroll
                            for (int h = 0; h < kPieces; ++h)
                                if (32 * hh + 16 * h < NCOLS)
                                    *reinterpret_cast<uint4 *>(dst + 32 * hh + 16 * h) =
                                        make_uint4(wq[h][0], wq[h][1], wq[h][2], wq[h][3]);
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);  // let copies in flight land
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------

static bool magic_exact2(unsigned d, unsigned long long max_x, unsigned *magic)
{
    const unsigned long long m = ((1ULL << 32) + d - 1) / d;
    if (m >= (1ULL << 32)) return false;
    *magic = (unsigned)m;
    const unsigned long long e = m * d - (1ULL << 32);  // umulhi(x, m) = x / d while x * e < 2^32
    return e == 0 || max_x < (1ULL << 32) / e;
}

static int rows_needed(const ConvRowsParams &q, int T)
{
    // grid positions a step's MMAs can touch: the last tile reads 128 rows plus the taps' reach
    return (T - 1) * q.rows_per_tile * q.grid_w + 128 + (q.taps - 1) * q.grid_w + (q.taps - 1);
}

static void conv_rows_shape(ConvRowsParams &q, int T)
{
    q.tiles_per_step = T;
    q.boxes_per_stage = (rows_needed(q, T) + q.box_rows - 1) / q.box_rows;
    q.stage_bytes = (int)(((size_t)q.boxes_per_stage * q.box_rows * q.row_bytes + 1023) & ~(size_t)1023);
}

// TMA boxes of a step's operand block: as few as the 256-row limit of a box allows, equal in size
// (a multiple of the eight rows of a swizzle atom), sized for max_tiles_per_step
static void conv_rows_box(ConvRowsParams &q)
{
    const int rows = rows_needed(q, q.max_tiles_per_step);
    const int boxes = (rows + 255) / 256;
    q.box_rows = (((rows + boxes - 1) / boxes) + 7) & ~7;
}

size_t conv_rows_smem_bytes(const ConvRowsParams &q0)
{
    ConvRowsParams q = q0;
    conv_rows_shape(q, q.max_tiles_per_step);
    const size_t b_bytes = (((size_t)q.taps * q.taps * q.n_cols * q.row_bytes) + 1023) & ~(size_t)1023;
    return 1024 + b_bytes + (size_t)kStages2 * q.stage_bytes;
}

// Does the kernel serve a conv with `taps` x `taps` stride-1 taps on a grid_h x grid_w grid of
// row_bytes-byte positions and n_total output channels?  Fills what does not depend on the call.
bool conv_rows_plan(int grid_h, int grid_w, int row_bytes, int taps, int n_total, long long max_batch,
                    ConvRowsParams *q)
{
    if ((row_bytes != 32 && row_bytes != 64 && row_bytes != 128) || taps < 1 || taps > 4 || n_total % 16 ||
        n_total < 16 || n_total > 64 || grid_w < taps || grid_h < taps || grid_w > 64)
        return false;
    const int S = 128 / grid_w;
    if (S * grid_w < 108) return false;  // too many idle rows per tile
    const long long rows = max_batch * grid_h;
    if (rows * grid_w + 512 >= (1LL << 31)) return false;
    memset(q, 0, sizeof(*q));
    if (!magic_exact2((unsigned)grid_w, 256, &q->ws_magic)) return false;
    if (!magic_exact2((unsigned)grid_h, (unsigned long long)rows + 256, &q->hs_magic)) return false;
    q->grid_h = grid_h;
    q->grid_w = grid_w;
    q->row_bytes = row_bytes;
    q->taps = taps;
    q->rows_per_tile = S;
    q->n_cols = n_total;
    // tiles per step: as many (up to 4) as leave kStages2 operand blocks beside the weights
    for (int T = 4; T >= 1; T /= 2) {
        q->max_tiles_per_step = T;
        conv_rows_box(*q);
        if (conv_rows_smem_bytes(*q) <= 200 * 1024) return true;
    }
    return false;
}

cudaError_t conv_rows_launch(const void *map_a, const void *map_b, const ConvRowsParams &q0, int batch,
                             int sm_count, cudaStream_t st)
{
    ConvRowsParams q = q0;
    q.batch = batch;
    const long long grid_rows = (long long)batch * q.grid_h;
    q.total_tiles = (int)((grid_rows + q.rows_per_tile - 1) / q.rows_per_tile);
    int T = q.max_tiles_per_step;
    while (T > 1 && (q.total_tiles + T - 1) / T < 2 * sm_count) T /= 2;
    conv_rows_shape(q, T);
    q.total_steps = (q.total_tiles + T - 1) / T;
    const int grid = q.total_steps < sm_count ? q.total_steps : sm_count;
    const size_t smem = conv_rows_smem_bytes(q0);
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads2);
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
    // (the requantiser is a template parameter, not a branch: both epilogues in one kernel cost time)
    if (q.n_cols == 64 && q.taps == 2 && q.row_bytes == 128)
        e = q.affine ? go(conv_rows_kernel<64, 2, 128, true>) : go(conv_rows_kernel<64, 2, 128, false>);
    else if (q.n_cols == 64 && q.taps == 3 && q.row_bytes == 64)
        e = q.affine ? go(conv_rows_kernel<64, 3, 64, true>) : go(conv_rows_kernel<64, 3, 64, false>);
    else
        e = q.affine ? (q.n_cols == 16 ? go(conv_rows_kernel<16, 0, 0, true>)
                        : q.n_cols == 32 ? go(conv_rows_kernel<32, 0, 0, true>)
                        : q.n_cols == 48 ? go(conv_rows_kernel<48, 0, 0, true>) : go(conv_rows_kernel<64, 0, 0, true>))
                     : (q.n_cols == 16 ? go(conv_rows_kernel<16, 0, 0, false>)
                        : q.n_cols == 32 ? go(conv_rows_kernel<32, 0, 0, false>)
                        : q.n_cols == 48 ? go(conv_rows_kernel<48, 0, 0, false>) : go(conv_rows_kernel<64, 0, 0, false>));
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace accerl
