// The Monitor's indicators and the per-state choice between two policies (Section 2.4).
//
// kl_kernel: KL(pi_original || pi_smaller) per state from two logit matrices (Eq. KL), one warp
// per state, lanes striding over the actions; kl_stats_kernel reduces the per-state values to
// their mean and maximum (the "KL mean" and "KL max" indicators) in one block, in a fixed order,
// so that the result does not depend on scheduling.  mix_select_kernel overwrites the original
// policy's outputs with the smaller policy's for the states whose selector draw falls below alpha
// (the linear-alpha strategy of Section 3.2: the Actor follows the small network with
// probability alpha).
#include <math.h>

#include "internal.h"

namespace accerl {

namespace {

__device__ __forceinline__ double warp_max(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Double arithmetic: where the two policies nearly agree the terms p (log p - log q) cancel, and
// the indicator runs at the Monitor's interval, not per environment step.
__global__ void __launch_bounds__(128)
kl_kernel(const float *__restrict__ zo_all, const float *__restrict__ zs_all, int B, int A,
          float *__restrict__ kl)
{
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= B) return;
    const float *zo = zo_all + row * A, *zs = zs_all + row * A;
    double mo = -INFINITY, ms = -INFINITY;
    for (int i = lane; i < A; i += 32) {
        mo = fmax(mo, (double)zo[i]);
        ms = fmax(ms, (double)zs[i]);
    }
    mo = warp_max(mo);
    ms = warp_max(ms);
    double so = 0.0, ss = 0.0;
    for (int i = lane; i < A; i += 32) {
        so += exp((double)zo[i] - mo);
        ss += exp((double)zs[i] - ms);
    }
    const double lseo = mo + log(warp_sum(so)), lses = ms + log(warp_sum(ss));
    double acc = 0.0;
    for (int i = lane; i < A; i += 32) {
        const double lpo = (double)zo[i] - lseo, lps = (double)zs[i] - lses, p = exp(lpo);
        if (p > 0.0) acc += p * (lpo - lps);
    }
    acc = warp_sum(acc);
    if (lane == 0) kl[row] = (float)acc;
}

// stats[0] = mean, stats[1] = max of kl[0..B)
__global__ void __launch_bounds__(1024) kl_stats_kernel(const float *__restrict__ kl, int B, float *stats)
{
    __shared__ double s_sum[1024];
    __shared__ float s_max[1024];
    double sum = 0.0;
    float mx = -INFINITY;
    for (int i = threadIdx.x; i < B; i += blockDim.x) {
        const float v = kl[i];
        sum += (double)v;
        mx = fmaxf(mx, v);
    }
    s_sum[threadIdx.x] = sum;
    s_max[threadIdx.x] = mx;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) {
            s_sum[threadIdx.x] += s_sum[threadIdx.x + o];
            s_max[threadIdx.x] = fmaxf(s_max[threadIdx.x], s_max[threadIdx.x + o]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        stats[0] = (float)(s_sum[0] / (double)B);
        stats[1] = s_max[0];
    }
}

struct MixOut {
    float *logits;
    int32_t *actions;
    float *logp, *value, *entropy;
};

__global__ void __launch_bounds__(256)
mix_select_kernel(const float *__restrict__ u_select, float alpha, int B, int A, MixOut dst, MixOut src,
                  uint8_t *__restrict__ use_smaller)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const bool pick = u_select[b] < alpha;
    if (use_smaller) use_smaller[b] = pick ? 1 : 0;
    if (!pick) return;
    for (int i = 0; i < A; ++i) dst.logits[(long long)b * A + i] = src.logits[(long long)b * A + i];
    dst.actions[b] = src.actions[b];
    dst.logp[b] = src.logp[b];
    if (dst.value) dst.value[b] = src.value[b];
    if (dst.entropy) dst.entropy[b] = src.entropy[b];
}

}  // namespace

}  // namespace accerl

using namespace accerl;

extern "C" accerl_status accerl_policy_kl(const float *logits_original_dev, const float *logits_smaller_dev,
                                          int32_t batch, int32_t n_actions, float *kl_dev,
                                          float *kl_mean_max_dev, void *cuda_stream)
{
    if (!logits_original_dev || !logits_smaller_dev || !kl_dev) {
        set_error("kl: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch < 1 || n_actions < 1 || n_actions > 1024) {
        set_error("kl: batch must be positive and n_actions in 1..1024");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (((uintptr_t)logits_original_dev | (uintptr_t)logits_smaller_dev | (uintptr_t)kl_dev |
         (uintptr_t)kl_mean_max_dev) & 3) {
        set_error("kl: misaligned pointer (4 bytes needed)");
        return ACCERL_ERR_INVALID_ARG;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const long long blocks = ((long long)batch * 32 + 127) / 128;
    kl_kernel<<<(unsigned)blocks, 128, 0, st>>>(logits_original_dev, logits_smaller_dev, batch, n_actions, kl_dev);
    ACCERL_CUDA_TRY(cudaGetLastError());
    if (kl_mean_max_dev) {
        kl_stats_kernel<<<1, 1024, 0, st>>>(kl_dev, batch, kl_mean_max_dev);
        ACCERL_CUDA_TRY(cudaGetLastError());
    }
    return ACCERL_OK;
}

extern "C" accerl_status accerl_policy_act_mixed(accerl_policy *smaller, accerl_policy *original,
                                                 const void *obs_dev, const float *uniforms_dev,
                                                 const float *select_uniforms_dev, float alpha,
                                                 int32_t batch, float *logits_dev, int32_t *actions_dev,
                                                 float *logp_dev, float *value_dev, float *entropy_dev,
                                                 uint8_t *use_smaller_dev, void *cuda_stream)
{
    if (!smaller || !original || !select_uniforms_dev) {
        set_error("act_mixed: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (smaller == original) {
        set_error("act_mixed: the two handles must differ (each owns the workspace its kernels write)");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (smaller->n_actions != original->n_actions || smaller->device != original->device ||
        smaller->in_kind != original->in_kind || smaller->in_c != original->in_c ||
        smaller->in_h != original->in_h || smaller->in_w != original->in_w) {
        set_error("act_mixed: the two policies must share device, observation shape and action count");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (!(alpha >= 0.f && alpha <= 1.f)) {
        set_error("act_mixed: alpha must lie in [0, 1]");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch < 1 || batch > smaller->max_batch || batch > original->max_batch) {
        set_error("act_mixed: batch %d outside 1..min(max_batch) = %d", batch,
                  smaller->max_batch < original->max_batch ? smaller->max_batch : original->max_batch);
        return batch < 1 ? ACCERL_ERR_INVALID_ARG : ACCERL_ERR_BATCH_TOO_LARGE;
    }
    if (value_dev && (smaller->n_out == smaller->n_actions || original->n_out == original->n_actions)) {
        set_error("act_mixed: value_dev given but a handle was created without ACCERL_FLAG_VALUE_HEAD");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (((uintptr_t)select_uniforms_dev & 3)) {
        set_error("act_mixed: misaligned pointer");
        return ACCERL_ERR_INVALID_ARG;
    }
    // the original policy writes the caller's buffers, the smaller one the handle's own
    accerl_status s = accerl_policy_act_ex(original, obs_dev, uniforms_dev, batch, logits_dev, actions_dev,
                                           logp_dev, value_dev, entropy_dev, cuda_stream);
    if (s != ACCERL_OK) return s;
    int prev = -1;
    cudaGetDevice(&prev);
    struct Restore {
        int prev;
        ~Restore() { if (prev >= 0) cudaSetDevice(prev); }
    } restore{prev};
    ACCERL_CUDA_TRY(cudaSetDevice(smaller->device));
    if (!smaller->mix_logits) {
        const size_t mb = (size_t)smaller->max_batch;
        const size_t sz[5] = {4 * mb * (size_t)smaller->n_actions, 4 * mb, 4 * mb, 4 * mb, 4 * mb};
        void *d[5];
        for (int i = 0; i < 5; ++i) {
            ACCERL_CUDA_TRY(cudaMalloc(&d[i], sz[i] + 256));
            smaller->owned.push_back(d[i]);
            smaller->workspace_bytes += sz[i] + 256;
        }
        smaller->mix_actions = (int32_t *)d[1];
        smaller->mix_logp = (float *)d[2];
        smaller->mix_value = (float *)d[3];
        smaller->mix_entropy = (float *)d[4];
        smaller->mix_logits = (float *)d[0];
    }
    s = accerl_policy_act_ex(smaller, obs_dev, uniforms_dev, batch, smaller->mix_logits, smaller->mix_actions,
                             smaller->mix_logp, value_dev ? smaller->mix_value : nullptr,
                             entropy_dev ? smaller->mix_entropy : nullptr, cuda_stream);
    if (s != ACCERL_OK) return s;
    MixOut dst{logits_dev, actions_dev, logp_dev, value_dev, entropy_dev};
    MixOut src{smaller->mix_logits, smaller->mix_actions, smaller->mix_logp, smaller->mix_value,
               smaller->mix_entropy};
    mix_select_kernel<<<(unsigned)((batch + 255) / 256), 256, 0, (cudaStream_t)cuda_stream>>>(
        select_uniforms_dev, alpha, batch, smaller->n_actions, dst, src, use_smaller_dev);
    ACCERL_CUDA_TRY(cudaGetLastError());
    return ACCERL_OK;
}
