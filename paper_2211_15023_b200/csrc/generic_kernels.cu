// Plain CUDA-core kernels for every layer kind: the path every network can take, and the
// cross-check for the tensor-core plans.  int8 x int8 -> int32 through dp4a on NHWC words.
#include "epilogue.cuh"
#include "internal.h"

namespace accerl {

// ---------------------------------------------------------------------------------------
// input stage
// ---------------------------------------------------------------------------------------

// uint8 NCHW -> int8 NHWC (channels padded to a multiple of 4).  One thread per output word;
// consecutive threads take consecutive pixels so the byte loads of a channel plane coalesce.
__global__ void ingest_u8_kernel(const uint8_t *__restrict__ obs, const int8_t *__restrict__ lut,
                                 int32_t *__restrict__ out, long long total_words, int C, int HW,
                                 int C4)
{
    __shared__ int8_t s_lut[256];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = lut[i];
    __syncthreads();
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    // idx = (n * C4 + c4) * HW + p  ->  output word (n * HW + p) * C4 + c4
    int p = (int)(idx % HW);
    long long t = idx / HW;
    int c4 = (int)(t % C4);
    long long n = t / C4;
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int c = c4 * 4 + j;
        if (c < C) {
            uint8_t u = obs[(n * C + c) * HW + p];
            word |= (uint32_t)(uint8_t)s_lut[u] << (8 * j);
        }
    }
    out[(n * HW + p) * C4 + c4] = (int32_t)word;
}

__global__ void ingest_f32_kernel(const float *__restrict__ obs, float s_input,
                                  int32_t *__restrict__ out, long long total_words, int D, int D4)
{
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total_words) return;
    int k4 = (int)(idx % D4);
    long long n = idx / D4;
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int k = k4 * 4 + j;
        if (k < D) word |= (uint32_t)(uint8_t)quantise_input(obs[n * D + k], s_input) << (8 * j);
    }
    out[idx] = (int32_t)word;
}

cudaError_t launch_ingest_u8(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int C,
                             int H, int W, int Cp, cudaStream_t st)
{
    long long total = (long long)B * H * W * (Cp / 4);
    int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    ingest_u8_kernel<<<(unsigned)blocks, threads, 0, st>>>(obs, lut, (int32_t *)out, total, C,
                                                           H * W, Cp / 4);
    return cudaGetLastError();
}

cudaError_t launch_ingest_f32(const float *obs, float s_input, int8_t *out, int B, int D, int Dp,
                              cudaStream_t st)
{
    long long total = (long long)B * (Dp / 4);
    int threads = 128;
    long long blocks = (total + threads - 1) / threads;
    ingest_f32_kernel<<<(unsigned)blocks, threads, 0, st>>>(obs, s_input, (int32_t *)out, total, D,
                                                            Dp / 4);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// direct convolution: one thread = one output pixel x 16 output channels
// ---------------------------------------------------------------------------------------

struct ConvArgs {
    const int32_t *in;    // NHWC words [B][H][W][C4]
    const int32_t *skip;  // NHWC words of the residual source, or null
    const int32_t *w;     // [tap][C4][oc_pad] words (4 input channels per word)
    const float *kscale, *bias;
    const int32_t *skip_mul;
    int8_t *out;          // NHWC bytes [B][OH][OW][out_cp]
    long long total_px;
    int H, W, C4, OH, OW, KH, KW, stride, pad, oc_pad, out_cp;
    float s_out;
    int relu_in, relu_out;
};

__global__ void __launch_bounds__(128) conv_dp4a_kernel(ConvArgs a)
{
    extern __shared__ int32_t s_w[];  // [tap][C4][16] for this block's channel group
    const int taps = a.KH * a.KW;
    const int oc0 = blockIdx.y * 16;
    for (int i = threadIdx.x; i < taps * a.C4 * 16; i += blockDim.x) {
        int j = i & 15, tc = i >> 4;
        s_w[i] = a.w[(long long)tc * a.oc_pad + oc0 + j];
    }
    __syncthreads();
    long long px = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (px >= a.total_px) return;
    int ox = (int)(px % a.OW);
    long long t = px / a.OW;
    int oy = (int)(t % a.OH);
    long long n = t / a.OH;

    int acc[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) acc[j] = 0;
    for (int ky = 0; ky < a.KH; ++ky) {
        int iy = oy * a.stride + ky - a.pad;
        if (iy < 0 || iy >= a.H) continue;
        for (int kx = 0; kx < a.KW; ++kx) {
            int ix = ox * a.stride + kx - a.pad;
            if (ix < 0 || ix >= a.W) continue;
            const int32_t *xin = a.in + ((n * a.H + iy) * a.W + ix) * a.C4;
            const int4 *wt = reinterpret_cast<const int4 *>(s_w + (ky * a.KW + kx) * a.C4 * 16);
            for (int c4 = 0; c4 < a.C4; ++c4) {
                int xv = __ldg(xin + c4);
                if (a.relu_in) xv = __vmaxs4(xv, 0);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int4 w4 = wt[c4 * 4 + j];
                    acc[4 * j + 0] = __dp4a(xv, w4.x, acc[4 * j + 0]);
                    acc[4 * j + 1] = __dp4a(xv, w4.y, acc[4 * j + 1]);
                    acc[4 * j + 2] = __dp4a(xv, w4.z, acc[4 * j + 2]);
                    acc[4 * j + 3] = __dp4a(xv, w4.w, acc[4 * j + 3]);
                }
            }
        }
    }
    // residual add in the int32 domain, then the float epilogue
    const int out_c4 = a.out_cp / 4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int oc = oc0 + 4 * j;
        if (oc < a.out_cp) {
            if (a.skip) {
                int sv = __ldg(a.skip + px * out_c4 + oc / 4);
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    acc[4 * j + b] += a.skip_mul[oc + b] * (int)(int8_t)(sv >> (8 * b));
            }
            uint32_t word = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                float y = epilogue_float(acc[4 * j + b], a.kscale[oc + b], a.bias[oc + b],
                                         a.relu_out);
                word |= (uint32_t)(uint8_t)requant(y, a.s_out) << (8 * b);
            }
            reinterpret_cast<uint32_t *>(a.out)[px * out_c4 + oc / 4] = word;
        }
    }
}

cudaError_t launch_conv_generic(const LayerPlan &L, const int8_t *in, const int8_t *skip,
                                int8_t *out, int B, cudaStream_t st)
{
    ConvArgs a;
    a.in = (const int32_t *)in;
    a.skip = (const int32_t *)skip;
    a.w = L.w_generic;
    a.kscale = L.kscale;
    a.bias = L.bias;
    a.skip_mul = L.skip_mul;
    a.out = out;
    a.total_px = (long long)B * L.out_h * L.out_w;
    a.H = L.in_h; a.W = L.in_w; a.C4 = L.in_cp / 4; a.OH = L.out_h; a.OW = L.out_w;
    a.KH = L.kh; a.KW = L.kw; a.stride = L.stride; a.pad = L.pad;
    a.oc_pad = L.oc_pad; a.out_cp = L.out_cp;
    a.s_out = L.s_out;
    a.relu_in = (L.flags & ACCERL_RELU_IN) != 0;
    a.relu_out = (L.flags & ACCERL_RELU_OUT) != 0;
    size_t smem = (size_t)L.kh * L.kw * a.C4 * 16 * sizeof(int32_t);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(conv_dp4a_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((unsigned)((a.total_px + 127) / 128), L.oc_pad / 16);
    conv_dp4a_kernel<<<grid, 128, smem, st>>>(a);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// fully connected: 64 x 64 output tile per block, K staged through shared memory
// ---------------------------------------------------------------------------------------

struct FcArgs {
    const int32_t *in;  // [B][K4] words
    const int32_t *w;   // [oc_pad][K4] words
    const float *kscale, *bias;
    int8_t *out;        // [B][out_cp] bytes
    float *logits;      // [B][out_c] when the layer produces logits
    int B, K4, oc_pad, out_cp, out_c;
    float s_out;
    int relu_in, relu_out;
};

__global__ void __launch_bounds__(256) fc_dp4a_kernel(FcArgs a)
{
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ int32_t As[BM][BK + 1];
    __shared__ int32_t Ws[BN][BK + 1];
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    const int row0 = blockIdx.x * BM, col0 = blockIdx.y * BN;
    int acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

    for (int k0 = 0; k0 < a.K4; k0 += BK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int idx = tid + i * 256, r = idx / BK, c = idx % BK;
            int row = row0 + r, col = col0 + r, k = k0 + c;
            int xv = (row < a.B && k < a.K4) ? __ldg(a.in + (long long)row * a.K4 + k) : 0;
            if (a.relu_in) xv = __vmaxs4(xv, 0);
            As[r][c] = xv;
            Ws[r][c] = (col < a.oc_pad && k < a.K4) ? __ldg(a.w + (long long)col * a.K4 + k) : 0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            int av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) av[i] = As[ty * 4 + i][kk];
#pragma unroll
            for (int j = 0; j < 4; ++j) bv[j] = Ws[tx * 4 + j][kk];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    const int oc = col0 + tx * 4;
    if (oc >= a.oc_pad) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int row = row0 + ty * 4 + i;
        if (row >= a.B) continue;
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float y = epilogue_float(acc[i][j], a.kscale[oc + j], a.bias[oc + j], a.relu_out);
            if (a.logits) {
                if (oc + j < a.out_c) a.logits[(long long)row * a.out_c + oc + j] = y;
            } else {
                word |= (uint32_t)(uint8_t)requant(y, a.s_out) << (8 * j);
            }
        }
        if (!a.logits && oc < a.out_cp)
            reinterpret_cast<uint32_t *>(a.out)[((long long)row * a.out_cp + oc) / 4] = word;
    }
}

cudaError_t launch_fc_generic(const LayerPlan &L, const int8_t *in, int8_t *out, float *logits,
                              int B, cudaStream_t st)
{
    FcArgs a;
    a.in = (const int32_t *)in;
    a.w = L.w_generic;
    a.kscale = L.kscale;
    a.bias = L.bias;
    a.out = out;
    a.logits = (L.flags & ACCERL_LOGITS) ? logits : nullptr;
    a.B = B;
    a.K4 = L.in_cp * L.in_h * L.in_w / 4;
    a.oc_pad = L.oc_pad; a.out_cp = L.out_cp; a.out_c = L.out_c;
    a.s_out = L.s_out;
    a.relu_in = (L.flags & ACCERL_RELU_IN) != 0;
    a.relu_out = (L.flags & ACCERL_RELU_OUT) != 0;
    dim3 grid((B + 63) / 64, (L.oc_pad + 63) / 64);
    fc_dp4a_kernel<<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// max-pool on NHWC words
// ---------------------------------------------------------------------------------------

__global__ void maxpool_kernel(const int32_t *__restrict__ in, int32_t *__restrict__ out,
                               long long total, int H, int W, int C4, int OH, int OW, int k,
                               int stride)
{
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    int c4 = (int)(idx % C4);
    long long t = idx / C4;
    int ox = (int)(t % OW);
    t /= OW;
    int oy = (int)(t % OH);
    long long n = t / OH;
    unsigned m = 0x80808080u;
    for (int ky = 0; ky < k; ++ky)
        for (int kx = 0; kx < k; ++kx) {
            int v = __ldg(in + ((n * H + oy * stride + ky) * W + ox * stride + kx) * C4 + c4);
            m = __vmaxs4(m, (unsigned)v);
        }
    out[idx] = (int)m;
}

cudaError_t launch_maxpool_generic(const LayerPlan &L, const int8_t *in, int8_t *out, int B,
                                   cudaStream_t st)
{
    int C4 = L.in_cp / 4;
    long long total = (long long)B * L.out_h * L.out_w * C4;
    maxpool_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        (const int32_t *)in, (int32_t *)out, total, L.in_h, L.in_w, C4, L.out_h, L.out_w, L.kh,
        L.stride);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// log-softmax + inverse-CDF sampling + behaviour log-prob
// ---------------------------------------------------------------------------------------

// Optional outputs of the sampler beside action and log-prob.  `z` rows are `pitch` floats apart
// and may hold one column more than there are actions: the state value V(s) (a policy with a value
// head), which takes no part in the softmax.  logits_out (rows of A floats) is written when the
// logits do not already sit where the caller wants them.
struct SampleExtras {
    int pitch;
    float *logits_out, *value, *entropy;
};

// A <= 32: a row occupies a power-of-two segment of a warp, one lane per action; max, sum and
// the running CDF are segment-wide shuffles, the bucket search is a ballot.
template <int WIDTH>
__global__ void sample_warp_kernel(const float *__restrict__ logits, const float *__restrict__ u,
                                   int B, int A, int32_t *__restrict__ actions,
                                   float *__restrict__ logp, const SampleExtras x)
{
    constexpr int ROWS_PER_WARP = 32 / WIDTH;
    const int lane = threadIdx.x & 31;
    const int seg = lane / WIDTH, sl = lane % WIDTH;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long row = warp * ROWS_PER_WARP + seg;
    const bool live = row < B && sl < A;
    float z = live ? logits[row * x.pitch + sl] : -INFINITY;
    if (live && x.logits_out) x.logits_out[row * A + sl] = z;
    if (x.value && row < B && sl == 0) x.value[row] = logits[row * x.pitch + A];
    float m = z;
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o, WIDTH));
    // The first maximal lane contributes exp(0) = 1 exactly; summing only the others and
    // taking log1p keeps log-probs near zero accurate to a few ulps of themselves.
    const unsigned seg_mask = (WIDTH == 32 ? 0xffffffffu : ((1u << WIDTH) - 1u)) << (seg * WIDTH);
    const unsigned ismax = __ballot_sync(0xffffffffu, live && z == m) & seg_mask;
    const int amax = ismax ? __ffs(ismax) - 1 - seg * WIDTH : 0;
    float e = (live && sl != amax) ? expf(z - m) : 0.f;
    float s = e;
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o, WIDTH);
    float lp = live ? (z - m) - log1pf(s) : 0.f;
    float p = live ? expf(lp) : 0.f;
    if (x.entropy) {  // H = -sum p log p over the segment
        float h = p > 0.f ? -p * lp : 0.f;
#pragma unroll
        for (int o = WIDTH / 2; o > 0; o >>= 1) h += __shfl_xor_sync(0xffffffffu, h, o, WIDTH);
        if (row < B && sl == 0) x.entropy[row] = h;
    }
    float cdf = p;  // inclusive scan within the segment
#pragma unroll
    for (int o = 1; o < WIDTH; o <<= 1) {
        float v = __shfl_up_sync(0xffffffffu, cdf, o, WIDTH);
        if (sl >= o) cdf += v;
    }
    float uu = row < B ? u[row] : 2.f;
    unsigned hit = __ballot_sync(0xffffffffu, live && uu < cdf);
    unsigned h = hit & seg_mask;
    int a = h ? (__ffs(h) - 1 - seg * WIDTH) : (A - 1);
    float lpa = __shfl_sync(0xffffffffu, lp, seg * WIDTH + a);
    if (row < B && sl == 0) {
        actions[row] = a;
        logp[row] = lpa;
    }
}

// any A: one warp per row, lanes stride over the actions
__global__ void sample_wide_kernel(const float *__restrict__ logits, const float *__restrict__ u,
                                   int B, int A, int32_t *__restrict__ actions,
                                   float *__restrict__ logp, const SampleExtras x)
{
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= B) return;
    const float *z = logits + row * x.pitch;
    if (x.logits_out)
        for (int i = lane; i < A; i += 32) x.logits_out[row * A + i] = z[i];
    if (x.value && lane == 0) x.value[row] = z[A];
    float m = -INFINITY;
    for (int i = lane; i < A; i += 32) m = fmaxf(m, z[i]);
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    int amax = A;  // first index that attains the maximum
    for (int i = lane; i < A; i += 32)
        if (z[i] == m) { amax = i; break; }
    for (int o = 16; o > 0; o >>= 1) amax = min(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    float s = 0.f;  // sum over all but the maximal term, which is exp(0) = 1
    for (int i = lane; i < A; i += 32)
        if (i != amax) s += expf(z[i] - m);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float l1p = log1pf(s), uu = u[row];
    if (x.entropy) {
        float h = 0.f;
        for (int i = lane; i < A; i += 32) {
            const float lp = (z[i] - m) - l1p, p = expf(lp);
            if (p > 0.f) h -= p * lp;
        }
        for (int o = 16; o > 0; o >>= 1) h += __shfl_xor_sync(0xffffffffu, h, o);
        if (lane == 0) x.entropy[row] = h;
    }
    float base = 0.f;
    int a = A - 1;
    bool found = false;
    for (int i0 = 0; i0 < A && !found; i0 += 32) {
        int i = i0 + lane;
        float p = i < A ? expf((z[i] - m) - l1p) : 0.f, cdf = p;
        for (int o = 1; o < 32; o <<= 1) {
            float v = __shfl_up_sync(0xffffffffu, cdf, o);
            if (lane >= o) cdf += v;
        }
        cdf += base;
        unsigned hit = __ballot_sync(0xffffffffu, i < A && uu < cdf);
        if (hit) {
            a = i0 + __ffs(hit) - 1;
            found = true;
        }
        base = __shfl_sync(0xffffffffu, cdf, 31);
    }
    if (lane == 0) {
        actions[row] = a;
        logp[row] = (z[a] - m) - l1p;
    }
}

// z: [B][pitch] floats (pitch = A, or A + 1 with a value column); see SampleExtras
cudaError_t launch_sample(const float *z, int pitch, const float *u, int B, int A, float *logits_out,
                          int32_t *actions, float *logp, float *value, float *entropy, cudaStream_t st)
{
    const int threads = 128;
    auto blocks_for = [&](int rows_per_warp) {
        long long warps = ((long long)B + rows_per_warp - 1) / rows_per_warp;
        return (unsigned)((warps * 32 + threads - 1) / threads);
    };
    SampleExtras x;
    x.pitch = pitch;
    x.logits_out = logits_out;
    x.value = value;
    x.entropy = entropy;
    if (A <= 2) sample_warp_kernel<2><<<blocks_for(16), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    else if (A <= 4) sample_warp_kernel<4><<<blocks_for(8), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    else if (A <= 8) sample_warp_kernel<8><<<blocks_for(4), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    else if (A <= 16) sample_warp_kernel<16><<<blocks_for(2), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    else if (A <= 32) sample_warp_kernel<32><<<blocks_for(1), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    else sample_wide_kernel<<<blocks_for(1), threads, 0, st>>>(z, u, B, A, actions, logp, x);
    return cudaGetLastError();
}

}  // namespace accerl
