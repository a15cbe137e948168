// Single-fma requantiser: the search, at create, for the per-channel constants.
//
// The requantiser q(acc) = clamp(rintf(relu?(fmaf((float)acc, k, b)) / s_out), -128, 127) is a
// non-decreasing step function of the int32 accumulator (k = s_in * s_w[c] > 0; every rounding
// in it is monotone).  So is a(acc) = relu?(clamp(rint(fmaf((float)acc, k2, b2)))) for k2 > 0.
// Two non-decreasing functions that agree on every integer of [lo, hi], with both already at the
// lowest code at lo and at 127 at hi, agree on all of int32.  The band [lo, hi] has a few hundred
// thousand integers, so the comparison is exhaustive and cheap.  (k2, b2) = (fl(k / s_out),
// fl(b / s_out)) is right for most channels; where a handful of accumulators near a rounding tie
// come out differently, neighbours of the pair are tried -- b2 in steps of 2^-21, k2 in ulps --
// until one agrees everywhere.  A layer all of whose channels have such a pair runs its epilogue
// with one fma per element instead of the three-step division; any other layer keeps that one.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "epilogue.cuh"
#include "internal.h"
#include "tc_gemm.h"

namespace accerl {

namespace {

constexpr int kKOffsets = 25;   // k2: 0, +1, -1, ... +12, -12 ulps
constexpr int kBOffsets = 49;   // b2: 0, +1, -1, ... +24, -24 steps of 2^-21
constexpr int kFitThreads = 256;
constexpr int kPerThread = 16;  // accumulators a thread compares between two votes
constexpr int kMaxBad = 16;

struct FitJob {
    float k, b;          // the channel's epilogue constants
    float k0, b0;        // fl(k / s_out), fl(b / s_out)
    long long lo, hi;    // band of accumulators to compare (inside int32)
    int check_lo, check_hi;  // 1: the band's end is no int32 limit, so both functions must be saturated there
};

struct FitResult {
    float k2, b2;
    int found, tries;
};

__device__ __forceinline__ int alternate(int i) { return (i & 1) ? (i + 1) / 2 : -(i / 2); }  // 0, 1, -1, 2, -2, ...

template <bool RELU>
__global__ void __launch_bounds__(kFitThreads) fit_affine_kernel(const FitJob *jobs, FitResult *results, float s_out)
{
    __shared__ long long bad[kMaxBad];  // accumulators on which an earlier candidate failed: tried first
    __shared__ int n_bad;
    const FitJob job = jobs[blockIdx.x];
    if (threadIdx.x == 0) n_bad = 0;
    __syncthreads();
    auto agree = [&](long long a, float k2, float b2) {
        return affine_code<RELU>((int)a, k2, b2) == exact_code(epilogue_float((int)a, job.k, job.b, false), s_out, RELU);
    };
    for (int cand = 0; cand < kKOffsets * kBOffsets; ++cand) {
        const float k2 = __uint_as_float(__float_as_uint(job.k0) + (unsigned)alternate(cand % kKOffsets));
        const float b2 = __fadd_rn(job.b0, __int2float_rn(alternate(cand / kKOffsets)) * 4.76837158203125e-7f);
        if (!(k2 > 0.f)) continue;  // uniform over the block
        // the accumulators that refuted earlier candidates, and the two ends of the band
        bool fail = false;
        const int known = min(n_bad, kMaxBad);
        if ((int)threadIdx.x < known) fail = !agree(bad[threadIdx.x], k2, b2);
        if (threadIdx.x == kFitThreads - 1) {
            if (job.check_lo && affine_code<RELU>((int)job.lo, k2, b2) != (RELU ? 0 : -128)) fail = true;
            if (job.check_hi && affine_code<RELU>((int)job.hi, k2, b2) != 127) fail = true;
        }
        if (__syncthreads_or(fail)) continue;
        // the whole band, a slice at a time
        bool refuted = false;
        for (long long base = job.lo; base <= job.hi && !refuted; base += (long long)kFitThreads * kPerThread) {
            long long first_bad = 0;
            bool any_bad = false;
            for (int j = 0; j < kPerThread; ++j) {
                const long long a = base + (long long)j * kFitThreads + threadIdx.x;
                if (a <= job.hi && !any_bad && !agree(a, k2, b2)) {
                    first_bad = a;
                    any_bad = true;
                }
            }
            if (any_bad) {
                const int slot = atomicAdd(&n_bad, 1);
                if (slot < kMaxBad) bad[slot] = first_bad;
            }
            refuted = __syncthreads_or(any_bad) != 0;
        }
        if (!refuted) {
            if (threadIdx.x == 0) results[blockIdx.x] = FitResult{k2, b2, 1, cand + 1};
            return;
        }
    }
    if (threadIdx.x == 0) results[blockIdx.x] = FitResult{job.k0, job.b0, 0, kKOffsets * kBOffsets};
}

// band of accumulators outside which both requantisers are saturated (or which int32 ends)
bool make_job(float k, float b, float s_out, bool relu, FitJob *job)
{
    if (!(k > 0.f) || !(s_out > 0.f) || !std::isfinite(k) || !std::isfinite(b) || !std::isfinite(s_out)) return false;
    const double dk = k, db = b, ds = s_out;
    const float k0 = (float)(dk / ds), b0 = (float)(db / ds);
    if (!(k0 > 0.f) || !std::isfinite(k0) || !std::isfinite(b0)) return false;
    // y = -2 s (ReLU: the code is 0 below) or -130 s at the low end, +130 s at the high end
    double lo = std::floor(((relu ? -2.0 : -130.0) * ds - db) / dk), hi = std::ceil((130.0 * ds - db) / dk);
    lo -= 16.0 + std::fabs(lo) * 0x1p-20;  // (float)acc is inexact above 2^24
    hi += 16.0 + std::fabs(hi) * 0x1p-20;
    job->k = k;
    job->b = b;
    job->k0 = k0;
    job->b0 = b0;
    job->check_lo = lo >= -2147483648.0;
    job->check_hi = hi <= 2147483647.0;
    job->lo = (long long)std::max(lo, -2147483648.0);
    job->hi = (long long)std::min(hi, 2147483647.0);
    // (bands of the networks here have 65 k - 350 k accumulators; the limit bounds the search time)
    return job->hi >= job->lo && job->hi - job->lo <= (1LL << 22);
}

}  // namespace

// For n columns with epilogue constants (k[i], b[i]) -- k[i] == 0 marks a padding column -- find the
// single-fma constants.  *ok = false (and k2, b2 untouched) when some column has none.
accerl_status fit_affine_requant(const float *k, const float *b, int n, float s_out, bool relu,
                                 std::vector<float> *k2, std::vector<float> *b2, bool *ok)
{
    *ok = false;
    std::vector<FitJob> jobs;
    std::vector<int> job_of(n, -1);
    for (int i = 0; i < n; ++i) {
        if (k[i] == 0.f && b[i] == 0.f) continue;  // padding column: the code is 0 either way
        int j = 0;
        for (; j < (int)jobs.size(); ++j)  // the columns of a multi-pixel row repeat the channels
            if (memcmp(&jobs[j].k, &k[i], 4) == 0 && memcmp(&jobs[j].b, &b[i], 4) == 0) break;
        if (j == (int)jobs.size()) {
            FitJob job;
            if (!make_job(k[i], b[i], s_out, relu, &job)) return ACCERL_OK;
            jobs.push_back(job);
        }
        job_of[i] = j;
    }
    std::vector<FitResult> res(jobs.size());
    if (!jobs.empty()) {
        FitJob *d_jobs = nullptr;
        FitResult *d_res = nullptr;
        ACCERL_CUDA_TRY(cudaMalloc(&d_jobs, jobs.size() * sizeof(FitJob)));
        cudaError_t e = cudaMalloc(&d_res, jobs.size() * sizeof(FitResult));
        if (e == cudaSuccess) e = cudaMemcpy(d_jobs, jobs.data(), jobs.size() * sizeof(FitJob), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) {
            if (relu) fit_affine_kernel<true><<<(unsigned)jobs.size(), kFitThreads>>>(d_jobs, d_res, s_out);
            else fit_affine_kernel<false><<<(unsigned)jobs.size(), kFitThreads>>>(d_jobs, d_res, s_out);
            e = cudaGetLastError();
        }
        if (e == cudaSuccess) e = cudaMemcpy(res.data(), d_res, jobs.size() * sizeof(FitResult), cudaMemcpyDeviceToHost);
        cudaFree(d_jobs);
        cudaFree(d_res);
        if (e != cudaSuccess) {
            set_error("fit_affine_requant: %s", cudaGetErrorString(e));
            return ACCERL_ERR_CUDA;
        }
        for (const FitResult &r : res)
            if (!r.found) return ACCERL_OK;
    }
    k2->assign(n, 0.f);
    b2->assign(n, 0.f);
    for (int i = 0; i < n; ++i)
        if (job_of[i] >= 0) {
            (*k2)[i] = res[job_of[i]].k2;
            (*b2)[i] = res[job_of[i]].b2;
        }
    *ok = true;
    return ACCERL_OK;
}

}  // namespace accerl
