// Small-batch latency path for all-FC policies on vector observations (the CartPole / LunarLander
// shaped networks at the paper's batch of 160 and up): the whole step -- input quantisation,
// every layer with its requantising epilogue, log-softmax, inverse-CDF sampling -- is ONE launch.
// At these sizes the step is bound by launch latency, not by arithmetic, so a chain of per-layer
// kernels would spend most of its time between kernels.
//
// A CTA owns kRows states.  Activations stay in shared memory as int8; thread o computes output
// o of the current layer for all of the CTA's rows with dp4a, reading the rows' words as
// shared-memory broadcasts and its weight words from global memory ([K/4][N] layout, coalesced).
#include <string.h>

#include "epilogue.cuh"
#include "internal.h"

namespace accerl {

namespace {
constexpr int kRows = 8;       // states per CTA
constexpr int kMaxWidth = 256; // widest layer (threads per CTA)
constexpr int kMaxLayers = 8;
}  // namespace

struct MlpFusedParams {
    int n_layers, in_dim, n_actions;
    float s_input;
    int k4[kMaxLayers];        // input words of layer l
    int n[kMaxLayers];         // outputs of layer l (multiple of 4 except the last)
    int relu[kMaxLayers];
    float s_out[kMaxLayers];
    const int32_t *w[kMaxLayers];     // [k4][n_pad] words, n_pad = round_up(n, 4)
    const float *kscale[kMaxLayers];  // [n]
    const float *bias[kMaxLayers];
    // parity taps (null without them): the quantised input and every hidden layer's int8 output
    // are also stored, rows of tap_in_pitch / tap_pitch[l] bytes
    int8_t *tap_in, *tap[kMaxLayers];
    int tap_in_pitch, tap_pitch[kMaxLayers];
};

__global__ void __launch_bounds__(kMaxWidth)
mlp_fused_kernel(const MlpFusedParams p, const float *__restrict__ obs, const float *__restrict__ u,
                 int B, float *__restrict__ logits, int32_t *__restrict__ actions,
                 float *__restrict__ logp, float *__restrict__ value, float *__restrict__ entropy)
{
    __shared__ __align__(16) int32_t act[2][kRows][kMaxWidth / 4];
    __shared__ float s_logits[kRows][32];
    const int tid = threadIdx.x, row0 = blockIdx.x * kRows;

    // input quantisation into act[0]
    const int k40 = p.k4[0];
    for (int i = tid; i < kRows * k40; i += blockDim.x) {
        const int r = i / k40, w4 = i - r * k40, row = row0 + r;
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = w4 * 4 + j;
            if (row < B && k < p.in_dim)
                word |= (uint32_t)(uint8_t)quantise_input(obs[(long long)row * p.in_dim + k], p.s_input)
                        << (8 * j);
        }
        act[0][r][w4] = (int32_t)word;
        if (p.tap_in && row < B && 4 * w4 < p.tap_in_pitch)
            *reinterpret_cast<uint32_t *>(p.tap_in + (long long)row * p.tap_in_pitch + 4 * w4) = word;
    }
    __syncthreads();

    int cur = 0;
    for (int l = 0; l < p.n_layers; ++l) {
        const int K4 = p.k4[l], N = p.n[l], n_pad = (N + 3) & ~3;
        const bool last = l == p.n_layers - 1;
        if (tid < N) {
            int acc[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r) acc[r] = 0;
            const int32_t *w = p.w[l] + tid;
            // weight words come from L2: keep eight loads in flight
            int k = 0;
            for (; k + 8 <= K4; k += 8) {
                int wv[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) wv[j] = __ldg(w + (long long)(k + j) * n_pad);
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int r = 0; r < kRows; ++r) acc[r] = __dp4a(act[cur][r][k + j], wv[j], acc[r]);
            }
            for (; k < K4; ++k) {
                const int wv = __ldg(w + (long long)k * n_pad);
#pragma unroll
                for (int r = 0; r < kRows; ++r) acc[r] = __dp4a(act[cur][r][k], wv, acc[r]);
            }
            const float ks = p.kscale[l][tid], bs = p.bias[l][tid];
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                const float y = epilogue_float(acc[r], ks, bs, p.relu[l] != 0);
                if (last) {  // columns [0, n_actions) are logits, a further one is the state value
                    s_logits[r][tid] = y;
                    if (row0 + r < B) {
                        if (tid < p.n_actions) logits[(long long)(row0 + r) * p.n_actions + tid] = y;
                        else if (value) value[row0 + r] = y;
                    }
                } else {
                    const int8_t code = requant(y, p.s_out[l]);
                    reinterpret_cast<int8_t *>(act[cur ^ 1][r])[tid] = code;
                    if (p.tap[l] && row0 + r < B) p.tap[l][(long long)(row0 + r) * p.tap_pitch[l] + tid] = code;
                }
            }
        } else if (!last && tid < n_pad) {
#pragma unroll
            for (int r = 0; r < kRows; ++r) reinterpret_cast<int8_t *>(act[cur ^ 1][r])[tid] = 0;
        }
        __syncthreads();
        cur ^= 1;
    }

    // sampling: one thread per row (at most 32 actions, all in registers / shared memory)
    if (tid < kRows && row0 + tid < B) {
        const int A = p.n_actions;
        const float *z = s_logits[tid];
        float m = z[0];
        int amax = 0;
        for (int i = 1; i < A; ++i)
            if (z[i] > m) {
                m = z[i];
                amax = i;
            }
        float s = 0.f;  // sum over all but the first maximal term, which is exp(0) = 1
        for (int i = 0; i < A; ++i)
            if (i != amax) s += expf(z[i] - m);
        const float l1p = log1pf(s), uu = u[row0 + tid];
        float cdf = 0.f, lp_a = 0.f, h = 0.f;
        int a = -1;
        for (int i = 0; i < A; ++i) {
            const float lp = (z[i] - m) - l1p, pi = expf(lp);
            if (pi > 0.f) h -= pi * lp;
            cdf += pi;
            if (a < 0 && uu < cdf) {
                a = i;
                lp_a = lp;
            }
        }
        if (a < 0) {
            a = A - 1;
            lp_a = (z[a] - m) - l1p;
        }
        actions[row0 + tid] = a;
        logp[row0 + tid] = lp_a;
        if (entropy) entropy[row0 + tid] = h;
    }
}

// Builds the fused plan when the policy qualifies; `used` says whether it did.
accerl_status build_mlp_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                             bool *used)
{
    *used = false;
    if (p->in_kind != ACCERL_IN_F32 || n_layers > kMaxLayers || p->n_out > 32) return ACCERL_OK;
    if (round_up(p->in_c, 4) > kMaxWidth) return ACCERL_OK;
    for (int i = 0; i < n_layers; ++i)
        if (layers[i].kind != ACCERL_FC || layers[i].out_c > kMaxWidth ||
            (layers[i].flags & ACCERL_RELU_IN))
            return ACCERL_OK;
    auto prm = std::make_shared<MlpFusedParams>();
    memset(prm.get(), 0, sizeof(MlpFusedParams));
    prm->n_layers = n_layers;
    prm->in_dim = p->in_c;
    prm->n_actions = p->n_actions;
    prm->s_input = p->s_input;
    int k_in = p->in_c;
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        const int K4 = round_up(k_in, 4) / 4, n_pad = round_up(d.out_c, 4);
        std::vector<int32_t> words((size_t)K4 * n_pad, 0);
        for (int o = 0; o < d.out_c; ++o)
            for (int k = 0; k < k_in; ++k)
                words[(size_t)(k / 4) * n_pad + o] |=
                    (int32_t)((uint32_t)(uint8_t)d.w[(size_t)o * k_in + k] << (8 * (k % 4)));
        void *dev = nullptr;
        accerl_status st = upload_bytes(p, words.data(), words.size() * 4, &dev);
        if (st != ACCERL_OK) return st;
        prm->w[i] = (const int32_t *)dev;
        prm->k4[i] = K4;
        prm->n[i] = d.out_c;
        prm->relu[i] = (d.flags & ACCERL_RELU_OUT) != 0;
        prm->s_out[i] = d.s_out;
        prm->kscale[i] = p->layers[i].kscale;
        prm->bias[i] = p->layers[i].bias;
        if ((p->flags & ACCERL_FLAG_KEEP_ACTIVATIONS) && i + 1 < n_layers) {
            prm->tap[i] = p->bufs[p->layers[i].out_buf].ptr;
            prm->tap_pitch[i] = p->layers[i].out_cp;
        }
        k_in = d.out_c;
    }
    if (p->flags & ACCERL_FLAG_KEEP_ACTIVATIONS) {
        prm->tap_in = p->bufs[p->layers[0].in_buf].ptr;
        prm->tap_in_pitch = p->in_cp;
    }
    p->mlp = prm;
    Step s;
    s.kind = Step::MLP_FUSED;
    s.kernel = "mlp_fused_kernel";
    s.covers = "ingest+layers 0-" + std::to_string(n_layers - 1) + "+sample";
    if (n_layers == 1) s.covers = "ingest+layer 0+sample";
    p->steps.assign(1, s);
    *used = true;
    return ACCERL_OK;
}

cudaError_t launch_mlp_fused(const accerl_policy *p, const float *obs, const float *u, int B,
                             float *logits, int32_t *actions, float *logp, float *value, float *entropy,
                             cudaStream_t st)
{
    const MlpFusedParams &prm = *p->mlp;
    mlp_fused_kernel<<<(B + kRows - 1) / kRows, kMaxWidth, 0, st>>>(prm, obs, u, B, logits, actions,
                                                                    logp, value, entropy);
    return cudaGetLastError();
}

}  // namespace accerl
