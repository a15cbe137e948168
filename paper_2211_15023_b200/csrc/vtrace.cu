// V-trace targets of the Corrector (Section 2.3, Eq. V-trace) and the policy-gradient advantage of
// Eq. A3C-V's first line, from the behaviour log-probs the Actor step emits.
//
// The definition is a double sum per start step s; it telescopes into the backward recursion
//   v_s - V(x_s) = delta_s + g_s c_s (v_{s+1} - V(x_{s+1})),   v_n = V(x_n) = bootstrap,
// which one thread runs for one trajectory, from the last step to the first.  Arrays are
// time-major [n][B], so the threads of a warp read consecutive floats at every step: the kernel
// moves 4 (5 with per-step discounts) input and 2 output floats per step and trajectory and is
// bound by HBM (by launch latency at the paper's batch sizes).  The recursion runs in double: its
// arithmetic is free next to the memory traffic, and the results then equal the double-precision
// definition up to the final rounding to float.
#include <math.h>

#include "internal.h"

namespace accerl {

namespace {

__global__ void __launch_bounds__(128)
vtrace_kernel(const float *__restrict__ logp_smaller, const float *__restrict__ logp_original,
              const float *__restrict__ rewards, const float *__restrict__ values,
              const float *__restrict__ bootstrap, const float *__restrict__ discounts, int n, int B,
              float gamma, float rho_hat, float c_hat, float *__restrict__ vs, float *__restrict__ adv)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    double v_next = (double)bootstrap[b];  // V(x_{t+1})
    double vs_next = v_next;               // v_{t+1}
    double carry = 0.0;                    // v_{t+1} - V(x_{t+1})
    // The recursion is sequential in t but its inputs are not: the loads of kChunk steps are issued
    // together (a rollout is one thread, so nothing else hides the memory latency).
    constexpr int kChunk = 8;
    for (int t1 = n - 1; t1 >= 0; t1 -= kChunk) {
        float lo[kChunk], ls[kChunk], rw[kChunk], vv[kChunk], dc[kChunk];
#pragma unroll
        for (int j = 0; j < kChunk; ++j) {
            const int t = t1 - j;
            const long long i = (long long)(t < 0 ? 0 : t) * B + b;
            lo[j] = logp_original[i];
            ls[j] = logp_smaller[i];
            rw[j] = rewards[i];
            vv[j] = values[i];
            dc[j] = discounts ? discounts[i] : gamma;
        }
#pragma unroll
        for (int j = 0; j < kChunk; ++j) {
            const int t = t1 - j;
            if (t < 0) break;
            const long long i = (long long)t * B + b;
            const double ratio = exp((double)lo[j] - (double)ls[j]);
            const double rho = fmin(ratio, (double)rho_hat), c = fmin(ratio, (double)c_hat);
            const double g = (double)dc[j];
            const double v = (double)vv[j], r = (double)rw[j];
            const double delta = rho * (r + g * v_next - v);
            carry = delta + g * c * carry;
            if (adv) adv[i] = (float)(rho * (r + g * vs_next - v));
            vs_next = v + carry;
            vs[i] = (float)vs_next;
            v_next = v;
        }
    }
}

}  // namespace

}  // namespace accerl

using namespace accerl;

extern "C" accerl_status accerl_vtrace(const float *logp_smaller_dev, const float *logp_original_dev,
                                       const float *rewards_dev, const float *values_dev,
                                       const float *bootstrap_dev, const float *discounts_dev,
                                       int32_t n_steps, int32_t batch, float gamma, float rho_hat,
                                       float c_hat, float *vs_dev, float *adv_dev, void *cuda_stream)
{
    if (!logp_smaller_dev || !logp_original_dev || !rewards_dev || !values_dev || !bootstrap_dev || !vs_dev) {
        set_error("vtrace: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (n_steps < 1 || batch < 1 || (long long)n_steps * batch >= (1LL << 40)) {
        set_error("vtrace: n_steps and batch must be positive (and n_steps * batch below 2^40)");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (!(gamma >= 0.f) || !(rho_hat > 0.f) || !(c_hat > 0.f) || !isfinite(gamma) || isnan(rho_hat) || isnan(c_hat)) {
        set_error("vtrace: gamma must be finite and non-negative, rho_hat and c_hat positive");
        return ACCERL_ERR_INVALID_ARG;
    }
    const uintptr_t all = (uintptr_t)logp_smaller_dev | (uintptr_t)logp_original_dev | (uintptr_t)rewards_dev |
                          (uintptr_t)values_dev | (uintptr_t)bootstrap_dev | (uintptr_t)discounts_dev |
                          (uintptr_t)vs_dev | (uintptr_t)adv_dev;
    if (all & 3) {
        set_error("vtrace: misaligned pointer (4 bytes needed)");
        return ACCERL_ERR_INVALID_ARG;
    }
    const int threads = batch >= 148 * 128 * 4 ? 128 : 32;  // few rollouts: spread them over the SMs
    vtrace_kernel<<<(unsigned)((batch + threads - 1) / threads), threads, 0, (cudaStream_t)cuda_stream>>>(
        logp_smaller_dev, logp_original_dev, rewards_dev, values_dev, bootstrap_dev, discounts_dev, n_steps,
        batch, gamma, rho_hat, c_hat, vs_dev, adv_dev);
    ACCERL_CUDA_TRY(cudaGetLastError());
    return ACCERL_OK;
}
