/*
 * CPU oracle for the Actor's int8 policy-inference path (TEST INFRASTRUCTURE).
 *
 * This file is a checker, not a product: it is slow on purpose, it is only
 * ever called from the tests, from the smoke check and from the benchmark's
 * CPU-baseline leg, and it shares no code with the CUDA library.
 *
 * What it computes.  The paper's Actor runs, for every environment step, a
 * forward pass of the Compressor's quantised policy on a batch of states and
 * samples an action per state (Introduction, Fig. 1: "Agent" time; Section
 * 2.2, paragraph "Parameter Quantization": int8 post-training quantisation
 * with Conv+ReLU / FC+ReLU fused into one layer).  The Corrector then needs
 * the behaviour probability of the sampled action (Section 2.3, Eq. V-trace:
 * rho_t and c_i are min(., pi_original / pi_smaller)).  The paper fixes no
 * arithmetic below that level; the arithmetic here is the one fixed requant
 * rule of this library,
 *
 *     q = clamp(rintf(fmaf((float)acc, s_in * s_w[c], b[c]) / s_out), -128, 127)
 *
 * with ReLU applied to the float before the clamp, int32 accumulation, and a
 * last layer that stops at the float (the logits).  Every function is the
 * definition written out as a naive loop nest, one output element at a time,
 * in NCHW / OIHW order.  The only parallelism is OpenMP over independent
 * states (or independent elements).
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math (fmaf is always
 * called explicitly; nothing may be contracted or reassociated).
 *
 * Parity status: every function below is pinned by the CPU tests (hand-worked
 * two-layer example, fp64 de-quantised forward, float64 library convolutions
 * on integer tensors, structural special cases, brute force for the sampler,
 * exhaustive ingest; entropy and KL against closed forms and scipy; V-trace
 * against the n-step return, the one-step TD target and a hand-worked rollout).  What stays unpinned: that this quantisation scheme is
 * the one the paper's authors ran -- the paper says only "PTQ" and "int8".
 */
#include <math.h>
#include <stdint.h>

static int8_t clamp_i8(float t)
{
    if (t < -128.0f) t = -128.0f;
    if (t > 127.0f) t = 127.0f;
    return (int8_t)t;
}

/* Input stage, frames: x = u / 255 (IEEE divide), q = clamp(rintf(x / s_input)). */
void oracle_ingest_u8(const uint8_t *u, int64_t n, float s_input, int8_t *q)
{
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i) {
        float x = (float)u[i] / 255.0f;
        q[i] = clamp_i8(rintf(x / s_input));
    }
}

/* Input stage, vectors: q = clamp(rintf(obs / s_input)). */
void oracle_ingest_f32(const float *obs, int64_t n, float s_input, int8_t *q)
{
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i)
        q[i] = clamp_i8(rintf(obs[i] / s_input));
}

/*
 * Convolution accumulators, zero padding:
 *   acc[n,oc,oy,ox] = sum_{ic,ky,kx} W[oc,ic,ky,kx] * X[n,ic,oy*s+ky-p,ox*s+kx-p]
 * relu_in != 0 replaces X by max(X, 0) first.
 */
void oracle_conv_acc(const int8_t *x, int B, int C, int H, int W, const int8_t *w, int OC,
                     int KH, int KW, int stride, int pad, int relu_in, int32_t *acc)
{
    const int OH = (H + 2 * pad - KH) / stride + 1;
    const int OW = (W + 2 * pad - KW) / stride + 1;
#pragma omp parallel for
    for (int n = 0; n < B; ++n)
        for (int oc = 0; oc < OC; ++oc)
            for (int oy = 0; oy < OH; ++oy)
                for (int ox = 0; ox < OW; ++ox) {
                    int32_t s = 0;
                    for (int ic = 0; ic < C; ++ic)
                        for (int ky = 0; ky < KH; ++ky)
                            for (int kx = 0; kx < KW; ++kx) {
                                int iy = oy * stride + ky - pad;
                                int ix = ox * stride + kx - pad;
                                if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
                                int32_t xv = x[(((int64_t)n * C + ic) * H + iy) * W + ix];
                                if (relu_in && xv < 0) xv = 0;
                                s += (int32_t)w[((oc * C + ic) * KH + ky) * KW + kx] * xv;
                            }
                    acc[(((int64_t)n * OC + oc) * OH + oy) * OW + ox] = s;
                }
}

/* Fully connected accumulators: acc[n,o] = sum_i W[o,i] * X[n,i]. */
void oracle_fc_acc(const int8_t *x, int B, int K, const int8_t *w, int N, int relu_in,
                   int32_t *acc)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n)
        for (int o = 0; o < N; ++o) {
            int32_t s = 0;
            for (int i = 0; i < K; ++i) {
                int32_t xv = x[(int64_t)n * K + i];
                if (relu_in && xv < 0) xv = 0;
                s += (int32_t)w[(int64_t)o * K + i] * xv;
            }
            acc[(int64_t)n * N + o] = s;
        }
}

/* Residual connection in the int32 domain: acc[n,c,p] += r[c] * skip[n,c,p]. */
void oracle_skip_add(int32_t *acc, const int8_t *skip, const int32_t *r, int B, int C, int HW)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < C; ++c)
            for (int p = 0; p < HW; ++p) {
                int64_t i = ((int64_t)n * C + c) * HW + p;
                acc[i] += r[c] * (int32_t)skip[i];
            }
}

/*
 * Epilogue float: y = fmaf((float)acc, k[c], b[c]) with k[c] = s_in * s_w[c]
 * rounded once to fp32; relu != 0 then takes max(y, 0).  This float is the
 * logit of a final layer, and the value whose max-abs the calibrator reads.
 */
void oracle_epilogue_float(const int32_t *acc, int B, int C, int HW, float s_in,
                           const float *s_w, const float *bias, int relu, float *y)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < C; ++c) {
            const float k = s_in * s_w[c];
            for (int p = 0; p < HW; ++p) {
                int64_t i = ((int64_t)n * C + c) * HW + p;
                float v = fmaf((float)acc[i], k, bias[c]);
                if (relu && v < 0.0f) v = 0.0f;
                y[i] = v;
            }
        }
}

/* Requantise: q = clamp(rintf(y / s_out), -128, 127), ties to even, IEEE divide. */
void oracle_requant(const float *y, int64_t n, float s_out, int8_t *q)
{
#pragma omp parallel for
    for (int64_t i = 0; i < n; ++i)
        q[i] = clamp_i8(rintf(y[i] / s_out));
}

/* Max-pool k x k, stride s, no padding, floor: per channel max over the window. */
void oracle_maxpool(const int8_t *x, int B, int C, int H, int W, int k, int stride, int8_t *out)
{
    const int OH = (H - k) / stride + 1;
    const int OW = (W - k) / stride + 1;
#pragma omp parallel for
    for (int n = 0; n < B; ++n)
        for (int c = 0; c < C; ++c)
            for (int oy = 0; oy < OH; ++oy)
                for (int ox = 0; ox < OW; ++ox) {
                    int8_t m = -128;
                    for (int ky = 0; ky < k; ++ky)
                        for (int kx = 0; kx < k; ++kx) {
                            int8_t v = x[(((int64_t)n * C + c) * H + oy * stride + ky) * W +
                                         ox * stride + kx];
                            if (v > m) m = v;
                        }
                    out[(((int64_t)n * C + c) * OH + oy) * OW + ox] = m;
                }
}

/*
 * Sampling and behaviour log-probability, in double from the fp32 logits:
 *   m = max z, lse = m + log sum exp(z - m), logp_i = z_i - lse,
 *   cdf_i = sum_{j<=i} exp(logp_j), action = first i with u < cdf_i, else A-1.
 * Outputs: logp_all [B,A] (double), action [B], logp_a [B] = (float)logp_action,
 * margin [B] = min_i |u - cdf_i| (how close the draw is to a bucket edge).
 */
void oracle_sample(const float *logits, int B, int A, const float *u, double *logp_all,
                   int32_t *action, float *logp_a, double *margin)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        const float *z = logits + (int64_t)n * A;
        double *lp = logp_all + (int64_t)n * A;
        double m = (double)z[0];
        for (int i = 1; i < A; ++i)
            if ((double)z[i] > m) m = (double)z[i];
        double s = 0.0;
        for (int i = 0; i < A; ++i) s += exp((double)z[i] - m);
        const double lse = m + log(s);
        for (int i = 0; i < A; ++i) lp[i] = (double)z[i] - lse;
        double cdf = 0.0, best = INFINITY;
        int a = -1;
        for (int i = 0; i < A; ++i) {
            cdf += exp(lp[i]);
            if (a < 0 && (double)u[n] < cdf) a = i;
            double d = fabs((double)u[n] - cdf);
            if (d < best) best = d;
        }
        if (a < 0) a = A - 1;
        action[n] = a;
        logp_a[n] = (float)lp[a];
        margin[n] = best;
    }
}

/*
 * Entropy of the action distribution, H(pi(.|s)) = -sum_i p_i log p_i, per state, in double
 * from the fp32 logits.  The paper uses it twice: as the regulariser of the distillation loss
 * (Section 2.2, Eq. KD, the term -beta H(pi_smaller)) and as one of the Monitor's indicators
 * (Section 2.4; Eq. advance lists "entropy" among the strategy's inputs).  Terms with p_i = 0
 * (exp underflow) contribute 0.
 */
void oracle_entropy(const float *logits, int B, int A, double *h)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        const float *z = logits + (int64_t)n * A;
        double m = (double)z[0];
        for (int i = 1; i < A; ++i)
            if ((double)z[i] > m) m = (double)z[i];
        double s = 0.0;
        for (int i = 0; i < A; ++i) s += exp((double)z[i] - m);
        const double lse = m + log(s);
        double acc = 0.0;
        for (int i = 0; i < A; ++i) {
            const double lp = (double)z[i] - lse, p = exp(lp);
            if (p > 0.0) acc -= p * lp;
        }
        h[n] = acc;
    }
}

/*
 * KL(pi_original || pi_smaller) = sum_a pi_original(a|x) log(pi_original(a|x) / pi_smaller(a|x))
 * per state (Section 2.4, Eq. KL: the Monitor's "KL mean" / "KL max" indicators are the mean and
 * the maximum of this over a batch), in double from two fp32 logit rows.
 */
void oracle_kl(const float *logits_original, const float *logits_smaller, int B, int A, double *kl)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        const float *zo = logits_original + (int64_t)n * A, *zs = logits_smaller + (int64_t)n * A;
        double mo = (double)zo[0], ms = (double)zs[0];
        for (int i = 1; i < A; ++i) {
            if ((double)zo[i] > mo) mo = (double)zo[i];
            if ((double)zs[i] > ms) ms = (double)zs[i];
        }
        double so = 0.0, ss = 0.0;
        for (int i = 0; i < A; ++i) {
            so += exp((double)zo[i] - mo);
            ss += exp((double)zs[i] - ms);
        }
        const double lseo = mo + log(so), lses = ms + log(ss);
        double acc = 0.0;
        for (int i = 0; i < A; ++i) {
            const double lpo = (double)zo[i] - lseo, lps = (double)zs[i] - lses, p = exp(lpo);
            if (p > 0.0) acc += p * (lpo - lps);
        }
        kl[n] = acc;
    }
}

/*
 * V-trace targets (Section 2.3, Eq. V-trace), written out as the definition: for every start
 * step s of a rollout of n steps,
 *
 *   v_s     = V(x_s) + sum_{t=s}^{n-1} (prod_{i=s}^{t-1} g_i c_i) delta_t
 *   delta_t = rho_t (r_t + g_t V(x_{t+1}) - V(x_t))
 *   rho_t   = min(rho_hat, pi_original / pi_smaller),   c_i = min(c_hat, pi_original / pi_smaller)
 *
 * with pi_original / pi_smaller = exp(logp_original - logp_smaller) of the action taken and
 * V(x_n) = bootstrap.  g_t is the constant gamma of the equation, or discounts[t] when a
 * per-step array is given (gamma times "episode goes on", the usual way of cutting the sums at
 * an episode end inside a rollout).  The sum of start step s runs to the end of the rollout.
 * Also returns the policy-gradient advantage of Eq. A3C-V's first line,
 *   adv_s = rho_s (r_s + g_s v_{s+1} - V(x_s)),  v_n = V(x_n).
 * All arrays are time-major [n][B]; everything is computed in double.
 */
void oracle_vtrace(const float *logp_smaller, const float *logp_original, const float *rewards,
                   const float *values, const float *bootstrap, const float *discounts, int n,
                   int B, float gamma, float rho_hat, float c_hat, double *vs, double *adv)
{
#pragma omp parallel for
    for (int b = 0; b < B; ++b) {
        for (int s = 0; s < n; ++s) {
            double sum = 0.0, prod = 1.0;
            for (int t = s; t < n; ++t) {
                const int64_t i = (int64_t)t * B + b;
                const double ratio = exp((double)logp_original[i] - (double)logp_smaller[i]);
                const double rho = ratio < (double)rho_hat ? ratio : (double)rho_hat;
                const double c = ratio < (double)c_hat ? ratio : (double)c_hat;
                const double g = discounts ? (double)discounts[i] : (double)gamma;
                const double v_next = t + 1 < n ? (double)values[i + B] : (double)bootstrap[b];
                const double delta = rho * ((double)rewards[i] + g * v_next - (double)values[i]);
                sum += prod * delta;
                prod *= g * c;
            }
            vs[(int64_t)s * B + b] = (double)values[(int64_t)s * B + b] + sum;
        }
        for (int s = 0; s < n; ++s) {
            const int64_t i = (int64_t)s * B + b;
            const double ratio = exp((double)logp_original[i] - (double)logp_smaller[i]);
            const double rho = ratio < (double)rho_hat ? ratio : (double)rho_hat;
            const double g = discounts ? (double)discounts[i] : (double)gamma;
            const double v_next = s + 1 < n ? vs[i + B] : (double)bootstrap[b];
            adv[i] = rho * ((double)rewards[i] + g * v_next - (double)values[i]);
        }
    }
}
