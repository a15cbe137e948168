// Micro-benchmark of the int8 tensor pipe (tcgen05.mma kind::i8, M = 128, K = 32 bytes per
// instruction): how many cycles one MMA of a given width N costs when the operands already sit in
// shared memory, and how that depends on the number of warps that issue.  It gives the measured
// denominator of the tensor-core roofline and the per-instruction costs the layer plans are built
// around (narrow tiles pay per instruction, not per multiply-accumulate).
//
// One CTA per SM: a 256 x 128-byte A tile (the MMA reads 128 rows of it, from row a_shift_rows on) and an N x 128-byte B tile (128-byte swizzle, K-major,
// contents arbitrary) are written once; then every issuing warp's elected lane issues
// `mmas_per_warp` MMAs back to back, walking the four 32-byte K steps of the tiles and rotating over
// its own accumulators in tensor memory, commits, and waits (bounded) for the pipe to drain.
#include "internal.h"
#include "tc_ptx.cuh"

namespace accerl {

namespace {

constexpr int kProbeMaxWarps = 4;

struct ProbeParams {
    int n, warps, mmas_per_warp, acc_per_warp;
    int overwrite;     // 1: the first MMA of every four overwrites its accumulator instead of adding to it
    int commit_every;  // 0, or: a tcgen05.commit (to a barrier nobody waits on) after every so many MMAs
    int a_shift_rows;  // the A operand starts this many rows into its tile (a row-shifted view)
    int layout;  // bytes of a swizzled K-major operand row (128, 64, 32), or 0: no swizzle, 16-byte K chunks in planes
    unsigned long long *cycles;  // [gridDim.x] cycles between the first issue and the drained pipe
    int *status;
};

__global__ void __launch_bounds__(32 * kProbeMaxWarps, 1) tc_probe_kernel(const ProbeParams p)
{
    extern __shared__ __align__(1024) uint8_t probe_smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)probe_smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t done_bar[kProbeMaxWarps], side_bar[kProbeMaxWarps];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *a_tile = smem, *b_tile = smem + 256 * 128;
    for (int i = threadIdx.x; i < (256 + p.n) * 128 / 4; i += blockDim.x)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x01010101u * (uint32_t)((i * 7 + 3) & 0x7f);
    if (threadIdx.x == 0) {
        for (int w = 0; w < kProbeMaxWarps; ++w) {
            mbar_init(smem_u32(&done_bar[w]), 1);
            mbar_init(smem_u32(&side_bar[w]), 1);
        }
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n >> 3) << 17) |
                           ((uint32_t)(128 >> 4) << 24);
    uint64_t adesc, bdesc;
    int ksteps;  // 32-byte K steps one operand row (or pair of planes) offers
    if (p.layout) {
        adesc = make_desc(smem_u32(a_tile) + (uint32_t)(p.a_shift_rows * p.layout), p.layout);
        bdesc = make_desc(smem_u32(b_tile), p.layout);
        ksteps = p.layout / 32;
    } else {
        // planes of [row][16 bytes]: 8-row groups 128 bytes apart, K chunks one plane apart
        auto planar = [](uint32_t addr, int rows) {
            return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)((rows * 16) >> 4) << 16) |
                   ((uint64_t)(128 >> 4) << 32) | ((uint64_t)1 << 46);
        };
        adesc = planar(smem_u32(a_tile) + (uint32_t)(p.a_shift_rows * 16), 256);
        bdesc = planar(smem_u32(b_tile), p.n);
        ksteps = 4;
    }
    const uint32_t a_step = p.layout ? 2u : (uint32_t)(2 * 256 * 16 >> 4), b_step = p.layout ? 2u : (uint32_t)(2 * p.n * 16 >> 4);
    long long t0 = 0;
    bool ok = true;
    if (warp < p.warps) {
        const uint32_t bar = smem_u32(&done_bar[warp]);
        const uint32_t acc0 = tmem_base + (uint32_t)(warp * p.acc_per_warp * p.n);
        __syncwarp();
        t0 = clock64();
        if (elect_one()) {
            int a = 0, until_commit = p.commit_every;
            for (int i = 0; i < p.mmas_per_warp; i += 4) {
                const uint32_t d = acc0 + (uint32_t)(a * p.n);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t kk = (uint32_t)(k & (ksteps - 1));
                    mma_i8(d, adesc + a_step * kk, bdesc + b_step * kk, idesc, p.overwrite ? (uint32_t)k : 1u);
                }
                if (++a == p.acc_per_warp) a = 0;
                if (p.commit_every && (until_commit -= 4) <= 0) {
                    mma_commit(smem_u32(&side_bar[warp]));
                    until_commit = p.commit_every;
                }
            }
            mma_commit(bar);
        }
        __syncwarp();
        ok = mbar_wait(bar, 0, &abort_flag, p.status, 1);
        ok = __all_sync(0xffffffffu, ok);
        const long long t1 = clock64();
        if (lane == 0 && ok) atomicMax(p.cycles + blockIdx.x, (unsigned long long)(t1 - t0));
    }
    if (abort_flag)
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u)
                     : "memory");
    }
}

}  // namespace

}  // namespace accerl

using namespace accerl;

extern "C" accerl_status accerl_tc_probe_i8(int32_t device, int32_t n, int32_t issuing_warps,
                                            int32_t mmas_per_warp, int32_t ctas, int32_t layout,
                                            int32_t a_shift_rows, int32_t commit_every, float *ms_out,
                                            float *cycles_per_mma_out)
{
    if (!ms_out || !cycles_per_mma_out) {
        set_error("tc_probe: null output");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (n < 16 || n > 256 || n % 16 || issuing_warps < 1 || issuing_warps > kProbeMaxWarps ||
        mmas_per_warp < 4 || mmas_per_warp > (1 << 20) || mmas_per_warp % 4 || ctas < 1 || ctas > 1024 ||
        issuing_warps * n > 512 || (layout != 0 && layout != 32 && layout != 64 && layout != 128) ||
        a_shift_rows < 0 || a_shift_rows > 128 || commit_every < 0 || (commit_every & 0xffff) % 4) {
        set_error("tc_probe: n in 16..256 (multiple of 16), 1..4 issuing warps with warps * n <= 512, "
                  "mmas_per_warp a multiple of 4 up to 2^20, 1..1024 CTAs, layout 0, 32, 64 or 128, a_shift_rows 0..128, commit_every a multiple of 4");
        return ACCERL_ERR_INVALID_ARG;
    }
    int ndev = 0, prev = -1;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        set_error("tc_probe: CUDA device %d not available", device);
        cudaGetLastError();
        return ACCERL_ERR_CUDA;
    }
    cudaGetDevice(&prev);
    struct Restore {
        int prev;
        ~Restore() { if (prev >= 0) cudaSetDevice(prev); }
    } restore{prev};
    ACCERL_CUDA_TRY(cudaSetDevice(device));
    cudaDeviceProp prop;
    ACCERL_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) {
        set_error("tc_probe: built for sm_100a only (device is sm_%d%d)", prop.major, prop.minor);
        return ACCERL_ERR_UNSUPPORTED;
    }
    ProbeParams q;
    q.n = n;
    q.warps = issuing_warps;
    q.mmas_per_warp = mmas_per_warp;
    q.acc_per_warp = 512 / (issuing_warps * n);
    q.layout = layout;
    q.a_shift_rows = a_shift_rows;
    q.commit_every = commit_every & 0xffff;
    q.overwrite = commit_every >> 16;
    void *dev = nullptr;
    const size_t bytes = (size_t)ctas * sizeof(unsigned long long) + 64;
    ACCERL_CUDA_TRY(cudaMalloc(&dev, bytes));
    struct Free {
        void *p;
        ~Free() { cudaFree(p); }
    } free_dev{dev};
    ACCERL_CUDA_TRY(cudaMemset(dev, 0, bytes));
    q.cycles = (unsigned long long *)dev;
    q.status = (int *)((char *)dev + (size_t)ctas * sizeof(unsigned long long));
    const size_t smem = 1024 + (size_t)(256 + n) * 128;
    ACCERL_CUDA_TRY(cudaFuncSetAttribute(tc_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    cudaEvent_t e0, e1;
    ACCERL_CUDA_TRY(cudaEventCreate(&e0));
    ACCERL_CUDA_TRY(cudaEventCreate(&e1));
    struct Events {
        cudaEvent_t a, b;
        ~Events() { cudaEventDestroy(a); cudaEventDestroy(b); }
    } events{e0, e1};
    float best = 0.f;
    for (int rep = 0; rep < 3; ++rep) {  // the first launch also loads the module
        ACCERL_CUDA_TRY(cudaMemset(dev, 0, bytes));
        ACCERL_CUDA_TRY(cudaEventRecord(e0, 0));
        tc_probe_kernel<<<ctas, 32 * kProbeMaxWarps, smem, 0>>>(q);
        ACCERL_CUDA_TRY(cudaGetLastError());
        ACCERL_CUDA_TRY(cudaEventRecord(e1, 0));
        ACCERL_CUDA_TRY(cudaEventSynchronize(e1));
        float ms = 0.f;
        ACCERL_CUDA_TRY(cudaEventElapsedTime(&ms, e0, e1));
        if (rep == 0 || ms < best) best = ms;
    }
    std::vector<unsigned long long> host((size_t)ctas + 8, 0);
    ACCERL_CUDA_TRY(cudaMemcpy(host.data(), dev, bytes, cudaMemcpyDeviceToHost));
    const int status = *(const int *)(host.data() + ctas);
    if (status) {
        set_error("tc_probe: a bounded wait gave up (status 0x%x)", status);
        return ACCERL_ERR_TIMEOUT;
    }
    double sum = 0;
    for (int i = 0; i < ctas; ++i) sum += (double)host[i];
    *ms_out = best;
    *cycles_per_mma_out = (float)(sum / ctas / ((double)mmas_per_warp * issuing_warps));
    return ACCERL_OK;
}
