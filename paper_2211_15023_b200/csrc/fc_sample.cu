// Last fully connected layer and the sampler in one launch: logits = fmaf((float)acc, k, b) for at
// most 32 actions, then log-softmax, inverse-CDF sampling and the behaviour log-prob of the drawn
// action.  The layer is tiny (K <= 1024, A <= 32), so a tensor-core launch plus a sampler launch
// spend most of their time starting and draining; here a warp owns two states at a time, lane j
// accumulates action j with dp4a from weights held in shared memory as [K/4][32] words, and the
// logits never leave registers before they are sampled (they are still written out: they are an
// output of the step).
#include <math.h>
#include <string.h>

#include <vector>

#include "epilogue.cuh"
#include "internal.h"

namespace accerl {

namespace {

constexpr int kFsWarps = 8;

// One row per warp, one lane per action: the arithmetic of sample_warp_kernel for a full-warp
// segment.  Every lane returns the drawn action and its log-prob.
template <bool ENTROPY>
__device__ __forceinline__ void warp_sample(float z, bool live, float uu, int A, int lane, int &a,
                                            float &lpa, float &h)
{
    if (!live) z = -INFINITY;
    float m = z;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    // the first maximal lane contributes exp(0) = 1 exactly: sum the others, take log1p
    const unsigned ismax = __ballot_sync(0xffffffffu, live && z == m);
    const int amax = ismax ? __ffs(ismax) - 1 : 0;
    float s = (live && lane != amax) ? expf(z - m) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float lp = live ? (z - m) - log1pf(s) : 0.f;
    float cdf = live ? expf(lp) : 0.f;  // inclusive scan
    if (ENTROPY) {  // H = -sum p log p
        h = cdf > 0.f ? -cdf * lp : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) h += __shfl_xor_sync(0xffffffffu, h, o);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float v = __shfl_up_sync(0xffffffffu, cdf, o);
        if (lane >= o) cdf += v;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, live && uu < cdf);
    a = hit ? __ffs(hit) - 1 : A - 1;
    lpa = __shfl_sync(0xffffffffu, lp, a);
}

// EXTRAS: the layer may have one output column more than actions, the state value V(s) (lane A;
// no part of the softmax), and the entropy of the action distribution may be asked for.
template <bool EXTRAS>
__global__ void __launch_bounds__(32 * kFsWarps)
fc_sample_kernel(const FcSampleParams q, const float *__restrict__ u, int B,
                 float *__restrict__ logits, int32_t *__restrict__ actions, float *__restrict__ logp,
                 float *__restrict__ value, float *__restrict__ entropy)
{
    extern __shared__ __align__(16) int32_t fs_smem[];
    const int K4 = q.k4, A = q.n_actions;
    int32_t *s_w = fs_smem;            // [K4][32]
    int32_t *s_x = fs_smem + K4 * 32;  // [warp][2][K4]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t *x0 = s_x + warp * 2 * K4, *x1 = x0 + K4;
    const bool live = lane < A;
    const bool has_col = EXTRAS ? lane < q.n_out : live;  // a column of the layer (action or value)
    const long long stride = (long long)gridDim.x * kFsWarps;
    long long pair = (long long)blockIdx.x * kFsWarps + warp;
    // The first rows, the weights and the scales are all fetched before anything waits: the
    // kernel is a chain of a few dependent memory round trips, not a throughput problem.
    uint4 r0[2], r1[2];  // K <= 1024: at most two 16-byte pieces of a row per lane
    auto fetch = [&](long long pr) {
        const long long row0 = 2 * pr, row1 = row0 + 1;
        const uint4 *g0 = reinterpret_cast<const uint4 *>(q.x + row0 * q.pitch);
        const uint4 *g1 = reinterpret_cast<const uint4 *>(q.x + row1 * q.pitch);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = lane + 32 * j;
            const bool in = i < K4 / 4 && row0 < B;
            r0[j] = in ? __ldg(g0 + i) : make_uint4(0, 0, 0, 0);
            r1[j] = (in && row1 < B) ? __ldg(g1 + i) : make_uint4(0, 0, 0, 0);
        }
    };
    // Programmatic dependent launch: the weights and scales do not depend on the previous launch,
    // so they are fetched while it drains; the rows it wrote are read after the wait.  (No early
    // trigger of its own: a next step's first layer that starts while this kernel still runs takes
    // its SMs' issue slots just to wait -- measured 194 against 177 us per Nature-CNN step.)
    const float ks = has_col ? q.kscale[lane] : 0.f, bs = has_col ? q.bias[lane] : 0.f;
    {
        const uint4 *gw = reinterpret_cast<const uint4 *>(q.w);
        uint4 *sw = reinterpret_cast<uint4 *>(s_w);
        for (int i = threadIdx.x; i < K4 * 8; i += blockDim.x) sw[i] = __ldg(gw + i);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    fetch(pair);
    __syncthreads();
    for (; 2 * pair < B; pair += stride) {
        const long long row0 = 2 * pair, row1 = row0 + 1;
        const bool has1 = row1 < B;
        const float u0 = u[row0], u1 = has1 ? u[row1] : 2.f;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = lane + 32 * j;
            if (i < K4 / 4) {
                reinterpret_cast<uint4 *>(x0)[i] = r0[j];
                reinterpret_cast<uint4 *>(x1)[i] = r1[j];
            }
        }
        __syncwarp();
        fetch(pair + stride);  // the next round's rows travel while this one computes
        int acc0 = 0, acc1 = 0;
#pragma unroll 4
        for (int k = 0; k < K4; k += 4) {
            const uint4 a0 = *reinterpret_cast<const uint4 *>(x0 + k);
            const uint4 a1 = *reinterpret_cast<const uint4 *>(x1 + k);
            const int w0 = s_w[k * 32 + lane], w1 = s_w[(k + 1) * 32 + lane];
            const int w2 = s_w[(k + 2) * 32 + lane], w3 = s_w[(k + 3) * 32 + lane];
            acc0 = __dp4a((int)a0.x, w0, acc0);
            acc1 = __dp4a((int)a1.x, w0, acc1);
            acc0 = __dp4a((int)a0.y, w1, acc0);
            acc1 = __dp4a((int)a1.y, w1, acc1);
            acc0 = __dp4a((int)a0.z, w2, acc0);
            acc1 = __dp4a((int)a1.z, w2, acc1);
            acc0 = __dp4a((int)a0.w, w3, acc0);
            acc1 = __dp4a((int)a1.w, w3, acc1);
        }
        __syncwarp();  // the staged rows are overwritten in the next round
        const float z0 = epilogue_float(acc0, ks, bs, false), z1 = epilogue_float(acc1, ks, bs, false);
        if (live) {
            logits[row0 * A + lane] = z0;
            if (has1) logits[row1 * A + lane] = z1;
        }
        if (EXTRAS && value && lane == A && A < q.n_out) {
            value[row0] = z0;
            if (has1) value[row1] = z1;
        }
        int a;
        float lpa, h = 0.f;
        if (EXTRAS && entropy) warp_sample<true>(z0, live, u0, A, lane, a, lpa, h);
        else warp_sample<false>(z0, live, u0, A, lane, a, lpa, h);
        if (lane == 0) {
            actions[row0] = a;
            logp[row0] = lpa;
            if (EXTRAS && entropy) entropy[row0] = h;
        }
        if (EXTRAS && entropy) warp_sample<true>(z1, live, u1, A, lane, a, lpa, h);
        else warp_sample<false>(z1, live, u1, A, lane, a, lpa, h);
        if (lane == 0 && has1) {
            actions[row1] = a;
            logp[row1] = lpa;
            if (EXTRAS && entropy) entropy[row1] = h;
        }
    }
}

}  // namespace

// Can layer i (the last one) run fused with the sampler?  Its input must be a plain [B][K] int8
// matrix written by a fully connected layer.
bool fc_sample_fits(const accerl_policy *p, const accerl_layer_desc *layers, int n_layers, int i)
{
    if (i != n_layers - 1 || i < 1) return false;
    const accerl_layer_desc &d = layers[i];
    const LayerPlan &L = p->layers[i];
    if (d.kind != ACCERL_FC || !(d.flags & ACCERL_LOGITS) || layers[i - 1].kind != ACCERL_FC) return false;
    if ((d.flags & ACCERL_RELU_IN) && !(layers[i - 1].flags & ACCERL_RELU_OUT)) return false;
    const int K = L.in_c;
    return L.in_h == 1 && L.in_w == 1 && L.in_cp == L.in_c && K % 16 == 0 && K >= 16 && K <= 1024 &&
           d.out_c <= 32;
}

// Packs the weights and fills the step; x is the layer's input matrix with rows of `pitch` bytes.
accerl_status build_fc_sample(accerl_policy *p, const accerl_layer_desc &d, int layer, const int8_t *x,
                              int pitch, Step *out)
{
    const LayerPlan &L = p->layers[layer];
    const int K = L.in_c, K4 = K / 4;
    std::vector<int32_t> words((size_t)K4 * 32, 0);
    for (int o = 0; o < d.out_c; ++o)
        for (int k = 0; k < K; ++k)
            words[(size_t)(k / 4) * 32 + o] |=
                (int32_t)((uint32_t)(uint8_t)d.w[(size_t)o * K + k] << (8 * (k % 4)));
    void *dev = nullptr;
    accerl_status st = upload_bytes(p, words.data(), words.size() * 4, &dev);
    if (st != ACCERL_OK) return st;
    FcSampleParams &q = p->fc_sample;
    q.x = x;
    q.pitch = pitch;
    q.k4 = K4;
    q.n_actions = p->n_actions;
    q.n_out = d.out_c;
    q.w = (const int32_t *)dev;
    q.kscale = L.kscale;
    q.bias = L.bias;
    out->kind = Step::FC_SAMPLE;
    out->layer = layer;
    out->kernel = "fc_sample_kernel";
    out->covers = "layer " + std::to_string(layer) + "+sample";
    return ACCERL_OK;
}

cudaError_t launch_fc_sample(const FcSampleParams &q, const float *u, int B, float *logits,
                             int32_t *actions, float *logp, float *value, float *entropy, int sm_count,
                             cudaStream_t st)
{
    const int per_block = 2 * kFsWarps;
    long long blocks = ((long long)B + per_block - 1) / per_block;
    if (blocks > 4LL * sm_count) blocks = 4LL * sm_count;
    const size_t smem = (size_t)q.k4 * 4 * (32 + 2 * kFsWarps);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(32 * kFsWarps);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool extras = value || entropy || q.n_out != q.n_actions;
    cudaError_t e = extras ? cudaLaunchKernelEx(&cfg, fc_sample_kernel<true>, q, u, B, logits, actions, logp, value, entropy)
                           : cudaLaunchKernelEx(&cfg, fc_sample_kernel<false>, q, u, B, logits, actions, logp,
                                                (float *)nullptr, (float *)nullptr);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace accerl
