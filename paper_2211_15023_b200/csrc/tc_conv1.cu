// First convolution of a frame policy with the input stage inside: uint8 NCHW frames with four
// channels, an 8 x 8 window and stride 4 (the first layer of the paper's Atari networks, table
// "network architecture and inference time") -> int8 activations in the next layer's layout.
//
// The conv is a 2 x 2 stride-1 conv on the space-to-depth(4) grid of the frame: one GEMM row per
// grid position (R, X), R = image * Hs + Y, 64 bytes of K per tap, four taps at row offsets
// 0, 1, Ws, Ws + 1 of ONE operand block in shared memory ("shifted rows").  What differs from the
// general contraction kernel:
//
// - No quantised copy of the frame ever exists, and no raw copy in shared memory either.
//   Converter warps read the frame words straight from global memory (one lane per grid position,
//   sixteen 4-byte loads: 4 channels x 4 image rows), quantise four bytes at a time and write the
//   position's 64-byte operand row.  K is ordered (channel, dy, dx) -- the order the bytes have in
//   the frame -- and the weights are permuted to match at create, so no byte is ever transposed.
//   Each converter warp owns two fixed row sets of every step; their next loads are in flight while
//   the current ones are converted.
// - A tile is S whole grid rows (S * Ws <= 128 GEMM rows), so a thread of the epilogue owns the
//   same (row, X) of every tile and decodes its output address with two multiplies.  A pipeline
//   step is T tiles; its operand block has one grid row more than it produces (the taps reach
//   into the next row), the only data converted twice.
// - MMA descriptors are computed in registers, eight MMAs per tile: the tensor pipe takes 40 cycles
//   for an M = 128, N <= 32 instruction (it is bound by reading the 4 KB operand from shared
//   memory).
// - Scales and biases are kernel parameters, read from the constant bank: with them in shared
//   memory the epilogue's broadcast loads queue behind the operand reads of the MMAs (measured:
//   113 against 94 us for the layer).
//
// Roles: warps 0..kMmaWarps1-1 issue MMAs (warp 0 owns tensor memory), the rest of warps 0..3 and
// warps kFirstExtraConv..kWarps-2 convert, the last warp prefetches frames into L2,
// warps 4..4+kEpiWarps-1 drain accumulators (warp w reads lane quarter w % 4).  Rings: kStages
// operand blocks (full / empty barriers), kAccSlots accumulators of 32 columns (one per tile).
// Every wait is bounded; a wait that gives up sets the status word and all roles leave.
#include <cuda.h>

#include <algorithm>
#include <type_traits>

#include "epilogue.cuh"
#include "internal.h"
#include "tc_conv1.h"
#include "tc_ptx.cuh"

namespace accerl {

namespace {

constexpr int kEpiWarps = 12;                       // three warpgroups
constexpr int kMmaWarps1 = 2;                       // issuing warps (tiles of a step in turn)
constexpr int kConvWarps = 9;                       // converter warps: two row sets of every step each
constexpr int kWarps = kMmaWarps1 + kConvWarps + kEpiWarps + 1;  // 24: the last one prefetches
constexpr int kFirstExtraConv = 4 + kEpiWarps;      // converters beyond warps kMmaWarps1..3 start here
constexpr int kPrefetchWarp = kWarps - 1;
constexpr int kPrefetchAhead = 3;                   // steps between a block being full and the prefetched one
constexpr int kThreads1 = 32 * kWarps;
constexpr int kStages = 3;
constexpr int kAccSlots = 16;  // x 32 columns = all 512 columns of tensor memory
constexpr int kMaxT = 4;

struct __align__(8) Bars1 {
    uint64_t full[kStages], empty[kStages];
    uint64_t acc_full[kAccSlots], acc_empty[kAccSlots];
    uint64_t b_ready;
    uint32_t tmem_base;
    int abort_flag;
    int conv_progress;  // steps the first converter warp has finished: paces the prefetch warp
};

// four frame bytes -> four codes by the fixed-point line q = min((u * mul + add) >> 24, 127)
template <bool CLAMP>
__device__ __forceinline__ uint32_t quantise_word_line(uint32_t w, uint32_t mul, uint32_t add)
{
    const uint32_t r0 = __byte_perm(w, 0, 0x4440) * mul + add, r1 = __byte_perm(w, 0, 0x4441) * mul + add;
    const uint32_t r2 = __byte_perm(w, 0, 0x4442) * mul + add, r3 = __byte_perm(w, 0, 0x4443) * mul + add;
    const uint32_t lo = __byte_perm(r0, r1, 0x0073), hi = __byte_perm(r2, r3, 0x0073);
    const uint32_t codes = __byte_perm(lo, hi, 0x5410);
    return CLAMP ? __vminu4(codes, 0x7f7f7f7fu) : codes;
}

// MODE 0: line without the min, 1: line with it, 2: the table is u >> 1
template <int MODE>
__device__ __forceinline__ uint32_t quantise_word(uint32_t w, uint32_t mul, uint32_t add)
{
    if (MODE == 2) return (w >> 1) & 0x7f7f7f7fu;
    return quantise_word_line<MODE == 1>(w, mul, add);
}

}  // namespace

// ATARI: the frame is 84 x 84 (a 21 x 21 grid, tiles of six grid rows); the divisions, strides and
// load offsets are then compile-time constants, which takes a third off the converters' instructions.
template <int NCOLS, int MODE, bool ATARI, bool AFFINE>
__global__ void __launch_bounds__(kThreads1, 1)
conv1_frames_kernel(const __grid_constant__ CUtensorMap map_b, const __grid_constant__ Conv1Params p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw1[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw1 + 1023) & ~(uintptr_t)1023);
    __shared__ Bars1 bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kBBytes = 4 * NCOLS * 64;  // four taps of [NCOLS][64 bytes]
    uint8_t *b_tiles = smem;
    uint8_t *stages = smem + ((kBBytes + 1023) & ~1023);
    const int stage_bytes = p.stage_bytes;
    volatile int *abort_flag = &bars.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), kConvWarps);
            mbar_init(smem_u32(&bars.empty[s]), kMmaWarps1);
        }
        for (int a = 0; a < kAccSlots; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);
        }
        mbar_init(smem_u32(&bars.b_ready), 1);
        bars.abort_flag = 0;
        bars.conv_progress = 0;
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
    // the next launch may set itself up while this grid drains; it waits for this grid's
    // completion before it reads what is written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int T = p.tiles_per_step, S = ATARI ? 6 : p.rows_per_tile, Ws = ATARI ? 21 : p.grid_w;
    const int Hs = ATARI ? 21 : p.grid_h;
    // x / Ws and x / Hs for the small non-negative values that occur
    auto div_ws = [&](unsigned x) { return ATARI ? x / 21u : __umulhi(x, p.ws_magic); };
    auto div_hs = [&](unsigned x) { return ATARI ? x / 21u : __umulhi(x, p.hs_magic); };
    const int my_steps = (int)blockIdx.x < p.total_steps
                             ? (p.total_steps - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const uint32_t full0 = smem_u32(&bars.full[0]), empty0 = smem_u32(&bars.empty[0]);
    const uint32_t acc_full0 = smem_u32(&bars.acc_full[0]), acc_empty0 = smem_u32(&bars.acc_empty[0]);

    if (warp < kMmaWarps1) {
        // ------------------------------------------------------------------ MMA issuers
        // (an issuing warp runs a hundred-odd instructions per tile beside the eight MMAs, and a warp
        // that shares its scheduler with five others issues one instruction every six to eight
        // cycles: one warp alone cannot keep the tensor pipe busy, so the tiles of a step go to
        // kMmaWarps1 warps in turn)
        if (warp == 0 && elect_one()) {
            mbar_expect_tx(smem_u32(&bars.b_ready), (uint32_t)kBBytes);
            for (int j = 0; j < 4; ++j)
                tma_load_2d(smem_u32(b_tiles) + j * NCOLS * 64, &map_b, 0, j * NCOLS, smem_u32(&bars.b_ready));
        }
        __syncwarp();
        bool ok = mbar_wait(smem_u32(&bars.b_ready), 0, abort_flag, p.status, 2);
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NCOLS >> 3) << 17) |
                               ((uint32_t)(128 >> 4) << 24);
        // 64-byte swizzled K-major rows: descriptor = constant upper word | (address >> 4)
        const uint64_t desc_hi = (uint64_t)(((uint32_t)(8 * 64) >> 4) | (1u << 14) | (4u << 29)) << 32;
        const uint32_t lo_flags = 1u << 16;
        const uint32_t b_lo = (smem_u32(b_tiles) >> 4) | lo_flags;
        const uint32_t tap_lo[4] = {0u, 4u, (uint32_t)(Ws * 4), (uint32_t)(Ws * 4 + 4)};  // 64-byte rows, >> 4
        for (int k = 0; k < my_steps && ok; ++k) {
            const int step = (int)blockIdx.x + k * (int)gridDim.x;
            const int s = k % kStages;
            const uint32_t par = (uint32_t)((k / kStages) & 1);
            ok = mbar_wait(full0 + 8 * s, par, abort_flag, p.status, 8);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t st_lo = ((smem_u32(stages) + (uint32_t)(s * stage_bytes)) >> 4) | lo_flags;
            for (int i = warp; i < T && ok; i += kMmaWarps1) {
                if (step * T + i >= p.total_tiles) break;
                const int seq = k * T + i, slot = seq % kAccSlots;  // the CTA's tiles in order
                const uint32_t slot_phase = (uint32_t)((seq / kAccSlots) & 1);
                ok = mbar_wait(acc_empty0 + 8 * slot, slot_phase ^ 1, abort_flag, p.status, 4);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (elect_one()) {
                    const uint32_t d = tmem_base + (uint32_t)(slot * 32);
                    const uint32_t a_lo = st_lo + (uint32_t)(i * S * Ws * 4);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks)
                            mma_i8(d, desc_hi | (a_lo + tap_lo[j] + 2 * ks),
                                   desc_hi | (b_lo + (uint32_t)(j * NCOLS * 4) + 2 * ks), idesc,
                                   (uint32_t)(j | ks));
                    mma_commit(acc_full0 + 8 * slot);
                }
                __syncwarp();
            }
            if (ok && elect_one()) mma_commit(empty0 + 8 * s);  // the block is free when these MMAs retire
            __syncwarp();
        }
    } else if (warp == kPrefetchWarp) {
        // ------------------------------------------------------------------ L2 prefetch
        // A converter warp has its loads in flight for one step only (two row sets fill its
        // registers), less than the memory latency under load.  This warp asks for the frame bytes of
        // the step kPrefetchAhead after the one just converted to be brought into L2, so that the
        // converters' loads find them there: whole image rows, up to eight runs of grid rows x four
        // planes per step, one bulk prefetch per lane.  (Issuing them from a converter warp made that
        // warp the slowest: the twelve-odd bulk operations take it about 900 cycles a step.)
        const int W = ATARI ? 84 : p.in_w, plane = ATARI ? 84 * 84 : p.in_plane;
        auto prefetch = [&](int k) {
            if (k >= my_steps) return;
            const int step = (int)blockIdx.x + k * (int)gridDim.x;
            const long long R0 = (long long)step * (T * S);
            const unsigned n0 = div_hs((unsigned)R0);
            const int seg = lane >> 2, c = lane & 3;  // run `seg` of the step lies in image n0 + seg
            const long long Ra = seg == 0 ? R0 : (long long)(n0 + seg) * Hs;
            long long Rb = (long long)(n0 + seg + 1) * Hs;
            Rb = Rb < R0 + T * S + 1 ? Rb : R0 + T * S + 1;
            Rb = Rb < p.total_grid_rows ? Rb : p.total_grid_rows;
            if (Ra >= Rb) return;
            const int Y = (int)(Ra - (long long)(n0 + seg) * Hs);
            const uint8_t *src = p.obs + ((size_t)(n0 + seg) * 4 + c) * plane + (size_t)(4 * Y) * W;
            const uint32_t bytes = (uint32_t)(Rb - Ra) * (uint32_t)(4 * W);  // 16-byte multiples: W % 4 == 0
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
        };
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int k = 1; k < kPrefetchAhead; ++k) prefetch(k);
        // paced by a counter, not by the barriers: a hint may fall behind or give up without harm
        volatile int *progress = &bars.conv_progress;
        for (int k = 0; k + kPrefetchAhead < my_steps; ++k) {
            int done = *progress;
            for (int polls = 0; done <= k && polls < (1 << 20) && !*abort_flag; ++polls) {
                __nanosleep(100);
                done = *progress;
            }
            if (done <= k) break;
            k = done - 1;  // the newest finished step, should this warp have fallen behind
            prefetch(k + kPrefetchAhead);
        }
    } else if (warp < 4 || warp >= kFirstExtraConv) {
        // ------------------------------------------------------------------ converters
        // A step's operand block has at most 2 * kConvWarps row sets of 32 grid positions; warp cw
        // owns sets cw and cw + kConvWarps of EVERY step, so a lane's two positions inside the block,
        // their operand-row addresses and swizzles are fixed for the whole kernel and only the image
        // and grid row behind them change from step to step.  While one set is quantised and written
        // the loads of the warp's next two sets travel (one set in flight exposes the full memory
        // latency per set).
        static_assert(kMmaWarps1 <= 4 && kConvWarps >= 1, "roles");
        const int cw = warp < 4 ? warp - kMmaWarps1 : warp - kFirstExtraConv + (4 - kMmaWarps1);  // 0 .. kConvWarps - 1
        const int step_rows = (T * S + 1) * Ws;            // grid positions a step's block holds
        const int W = ATARI ? 84 : p.in_w, plane = ATARI ? 84 * 84 : p.in_plane;
        const int posA = cw * 32 + lane, posB = (cw + kConvWarps) * 32 + lane;
        const bool vA = posA < step_rows, vB = posB < step_rows;
        const int RlA = (int)div_ws((unsigned)posA), XA = posA - RlA * Ws;
        const int RlB = (int)div_ws((unsigned)posB), XB = posB - RlB * Ws;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // loads of one position's sixteen words; never predicated: a position beyond the last image or
        // the last step reads the first image's bytes instead (its row is no output), which takes the
        // sixteen selects out of the loop (86 against 89.5 us for the layer)
        auto load = [&](uint32_t (&w)[16], int k, int Rl, int X, bool v) {
            // (32-bit row arithmetic: the plan has checked that batch * grid_h + 64 < 2^31)
            const unsigned R = (unsigned)(((int)blockIdx.x + k * (int)gridDim.x) * (T * S) + Rl);
            const bool in = v && k < my_steps && R < (unsigned)p.total_grid_rows;
            const unsigned n = div_hs(R);
            const int Y = (int)(R - n * (unsigned)Hs);
            const uint8_t *src = p.obs + (in ? (size_t)n * (size_t)(4 * plane) + (size_t)(4 * Y * W + 4 * X) : (size_t)0);
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int dy = 0; dy < 4; ++dy)
                    w[4 * c + dy] = __ldg(reinterpret_cast<const uint32_t *>(src + (size_t)c * plane + dy * W));
        };
        // quantise one set and write its operand rows: four 16-byte pieces under the 64-byte swizzle,
        // at 32-bit shared-memory addresses whose per-thread parts (off[c]) are computed once
        auto store = [&](const uint32_t (&w)[16], uint32_t block, const uint32_t (&off)[4], bool v) {
            if (!v) return;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(block + off[c]),
                             "r"(quantise_word<MODE>(w[4 * c], p.ingest_mul, p.ingest_add)),
                             "r"(quantise_word<MODE>(w[4 * c + 1], p.ingest_mul, p.ingest_add)),
                             "r"(quantise_word<MODE>(w[4 * c + 2], p.ingest_mul, p.ingest_add)),
                             "r"(quantise_word<MODE>(w[4 * c + 3], p.ingest_mul, p.ingest_add))
                             : "memory");
        };
        uint32_t offA[4], offB[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            offA[c] = (uint32_t)(posA * 64 + ((c ^ ((posA >> 1) & 3)) << 4));
            offB[c] = (uint32_t)(posB * 64 + ((c ^ ((posB >> 1) & 3)) << 4));
        }
        const uint32_t stages_s = smem_u32(stages);
        uint32_t wa[16], wb[16];
        load(wa, 0, RlA, XA, vA);
        load(wb, 0, RlB, XB, vB);
        bool ok = true;
        for (int k = 0; k < my_steps && ok; ++k) {
            const int s = k % kStages;
            ok = mbar_wait(empty0 + 8 * s, (uint32_t)(((k / kStages) & 1) ^ 1), abort_flag, p.status, 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t block = stages_s + (uint32_t)(s * stage_bytes);
            store(wa, block, offA, vA);
            load(wa, k + 1, RlA, XA, vA);
            store(wb, block, offB, vB);
            load(wb, k + 1, RlB, XB, vB);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(full0 + 8 * s);
                if (cw == 0) *(volatile int *)&bars.conv_progress = k + 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - 4, wg = ew >> 2, q = warp & 3;
        constexpr int kGroups = kEpiWarps / 4;
        const int r = q * 32 + lane;  // this thread's row of every tile
        const int Rl = (int)div_ws((unsigned)r), X = r - Rl * Ws;
        const int sh = p.out_s2d_log2, smask = (1 << sh) - 1;
        const bool row_ok = r < S * Ws && X < p.out_w;
        const int x_off = (X >> sh) * p.out_pitch + (X & smask) * p.n_total;
        const float s_out = p.s_out, inv_s_out = p.inv_s_out;
        asm volatile("griddepcontrol.wait;" ::: "memory");
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
                const uint32_t apar = (uint32_t)((seq / kAccSlots) & 1);
                ok = mbar_wait(acc_full0 + 8 * slot, apar, abort_flag, p.status, 16);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(slot * 32);
                int acc[NCOLS / 16][16];
#pragma unroll
                for (int h = 0; h < NCOLS / 16; ++h) tmem_ld16(taddr + 16 * h, acc[h]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty0 + 8 * slot);
                const unsigned R = (unsigned)(tile * S + Rl);
                const unsigned n = div_hs(R);
                const int Y = (int)(R - n * (unsigned)Hs);
                const bool valid = row_ok && Y < p.out_h && (int)n < p.batch;
                int8_t *dst = p.out + (size_t)(n * (unsigned)p.out_rows_per_image + (unsigned)((Y >> sh) * p.out_grid_w)) *
                                          (size_t)p.out_pitch +
                              (((Y & smask) << sh) * p.n_total + x_off);
                uint32_t wq[NCOLS / 16][4];
#pragma unroll
                for (int h = 0; h < NCOLS / 16; ++h) {
                    float ks[16], bs[16];
#pragma unroll
                    for (int g = 0; g < 4; ++g) {  // kernel parameters: 16-byte reads from the constant bank
                        const float4 kv = *reinterpret_cast<const float4 *>(&p.ks[16 * h + 4 * g]);
                        const float4 bv = *reinterpret_cast<const float4 *>(&p.bs[16 * h + 4 * g]);
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
                if (valid) {  // a position's channels are contiguous: 16 bytes, or 32 in one store
                    if constexpr (NCOLS == 32) stg32(dst, wq[0], wq[1]);
                    else *reinterpret_cast<uint4 *>(dst) = make_uint4(wq[0][0], wq[0][1], wq[0][2], wq[0][3]);
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

static bool magic_exact(unsigned d, unsigned long long max_x, unsigned *magic)
{
    const unsigned long long m = ((1ULL << 32) + d - 1) / d;
    if (m >= (1ULL << 32)) return false;
    *magic = (unsigned)m;
    const unsigned long long e = m * d - (1ULL << 32);  // umulhi(x, m) = x / d while x * e < 2^32
    return e == 0 || max_x < (1ULL << 32) / e;
}

// Does the dedicated kernel serve this first layer?  Fills everything of `q` that does not
// depend on the call's batch or pointers.
bool conv1_plan(const accerl_layer_desc &d, int in_h, int in_w, long long max_batch, int n_total,
                int ingest_mode, Conv1Params *q)
{
    if (d.kind != ACCERL_CONV2D || d.in_c != 4 || d.kh != 8 || d.kw != 8 || d.stride != 4 || d.pad != 0 ||
        d.skip_from >= 0 || in_h % 4 || in_w % 4 || (n_total != 16 && n_total != 32) || d.out_c != n_total)
        return false;
    const int Hs = in_h / 4, Ws = in_w / 4;
    if (Ws < 2 || Ws > 64 || Hs < 2) return false;
    const int S = 128 / Ws;
    if (S * Ws < 112) return false;  // too many idle rows per tile
    const long long rows = max_batch * Hs;
    if (rows + 64 >= (1LL << 31) || rows * Ws >= (1LL << 31)) return false;  // 32-bit row and output-row indices
    memset(q, 0, sizeof(*q));
    if (!magic_exact((unsigned)Ws, (unsigned long long)(kMaxT * S + 2) * Ws + 64, &q->ws_magic)) return false;
    if (!magic_exact((unsigned)Hs, (unsigned long long)rows + 256, &q->hs_magic)) return false;
    q->in_w = in_w;
    q->in_plane = in_h * in_w;
    q->grid_h = Hs;
    q->grid_w = Ws;
    q->rows_per_tile = S;
    q->n_cols = n_total;
    q->ingest_mode = ingest_mode;
    // positions a step's MMAs can touch: (T - 1) * S * Ws + 127 + Ws + 1, plus one for the count
    if (((kMaxT * S + 1) * Ws + 31) / 32 > 2 * kConvWarps) return false;  // two row sets per converter warp and step
    q->stage_bytes = (((kMaxT - 1) * S * Ws + 128 + Ws + 1) * 64 + 1023) & ~1023;
    return true;
}

size_t conv1_smem_bytes(const Conv1Params &q)
{
    return 1024 + (((size_t)4 * q.n_cols * 64 + 1023) & ~(size_t)1023) + (size_t)kStages * q.stage_bytes;
}

cudaError_t conv1_launch(const void *map_b, const Conv1Params &q0, int batch, const uint8_t *obs,
                         int sm_count, cudaStream_t st)
{
    Conv1Params q = q0;
    q.obs = obs;
    q.batch = batch;
    q.total_grid_rows = (long long)batch * q.grid_h;
    q.total_tiles = (int)((q.total_grid_rows + q.rows_per_tile - 1) / q.rows_per_tile);
    // tiles per step: four, fewer while that leaves SMs without work
    int T = kMaxT;
    while (T > 1 && (q.total_tiles + T - 1) / T < 2 * sm_count) T /= 2;
    q.tiles_per_step = T;
    q.total_steps = (q.total_tiles + T - 1) / T;
    const int grid = q.total_steps < sm_count ? q.total_steps : sm_count;
    const size_t smem = conv1_smem_bytes(q);
    auto go = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kThreads1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, *(const CUtensorMap *)map_b, q);
    };
    const bool atari = q.in_w == 84 && q.in_plane == 84 * 84;
    // (the requantiser is a template parameter, not a branch: with both epilogues in one kernel the
    // layer measured 4 to 7 us slower)
    auto pick = [&](auto ncols, auto is_atari) -> cudaError_t {
        constexpr int N = decltype(ncols)::value;
        constexpr bool A = decltype(is_atari)::value;
        if (q.affine)
            return q.ingest_mode == 2 ? go(conv1_frames_kernel<N, 2, A, true>)
                   : q.ingest_mode == 1 ? go(conv1_frames_kernel<N, 1, A, true>) : go(conv1_frames_kernel<N, 0, A, true>);
        return q.ingest_mode == 2 ? go(conv1_frames_kernel<N, 2, A, false>)
               : q.ingest_mode == 1 ? go(conv1_frames_kernel<N, 1, A, false>) : go(conv1_frames_kernel<N, 0, A, false>);
    };
    cudaError_t e;
    if (q.n_cols == 32)
        e = atari ? pick(std::integral_constant<int, 32>(), std::true_type()) : pick(std::integral_constant<int, 32>(), std::false_type());
    else
        e = atari ? pick(std::integral_constant<int, 16>(), std::true_type()) : pick(std::integral_constant<int, 16>(), std::false_type());
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace accerl
