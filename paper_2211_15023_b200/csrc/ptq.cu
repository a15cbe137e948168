// Post-training quantisation on the device (Section 2.2, paragraphs "Parameter Quantization" and
// "Structured Pruning"): accerl_policy_create_fp32 takes the fp32 network the Learner trains and a
// calibration batch, and does what the Compressor's quantiser does before it hands the Actor a
// policy -- optional 2:4 pruning, symmetric int8 weights with one scale per output channel
// (max|w| / 127), one scale per activation tensor (max-abs of the epilogue float over the
// calibration batch, pushed through the already quantised preceding layers), the integer
// multipliers of the residual adds -- and then builds the handle with accerl_policy_create.
//
// This is create-time work: the kernels are plain (one thread per output element, NCHW int8
// activations, int32 accumulators kept in memory between the passes of a layer) and every result
// is order-independent (integer sums, maxima), so the scales and codes are the same bits whatever
// the launch shape.  The Actor step itself never runs these kernels.
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "internal.h"

namespace accerl {

namespace {

__device__ __forceinline__ void atomic_max_nonneg(float *addr, float v)
{
    atomicMax(reinterpret_cast<int *>(addr), __float_as_int(v));  // v >= 0: the bit patterns order like the values
}

// 2:4 pruning along K = (kh, kw, c_in), c_in fastest: of every four consecutive K positions keep
// the two of largest |w| (the lower index wins a tie), zero the others.  In place, OIHW.
__global__ void prune24_kernel(float *w, int oc, int ic, int kh, int kw)
{
    const long long groups = (long long)oc * kh * kw * ic / 4;
    const long long gidx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gidx >= groups) return;
    const int per_oc = kh * kw * ic / 4;
    const int o = (int)(gidx / per_oc);
    const int k0 = (int)(gidx - (long long)o * per_oc) * 4;
    float v[4];
    long long at[4];
    for (int j = 0; j < 4; ++j) {
        const int k = k0 + j, c = k % ic, t = k / ic, x = t % kw, y = t / kw;
        at[j] = (((long long)o * ic + c) * kh + y) * kw + x;
        v[j] = w[at[j]];
    }
    // rank of element j: how many others come before it in a stable sort by decreasing |w|
    for (int j = 0; j < 4; ++j) {
        int before = 0;
        for (int i = 0; i < 4; ++i)
            if (i != j && (fabsf(v[i]) > fabsf(v[j]) || (fabsf(v[i]) == fabsf(v[j]) && i < j))) ++before;
        if (before >= 2) w[at[j]] = 0.f;
    }
}

// one block per output channel: s_w = max|w| / 127 (1 for an all-zero row), q = clip(rint(w / s_w))
__global__ void quantise_weights_kernel(const float *w, int K, float *s_w, int8_t *q)
{
    __shared__ float red[256];
    const int o = blockIdx.x;
    const float *row = w + (long long)o * K;
    float m = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) m = fmaxf(m, fabsf(row[k]));
    red[threadIdx.x] = m;
    __syncthreads();
    for (int s = blockDim.x / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + s]);
        __syncthreads();
    }
    const float s = red[0] > 0.f ? __fdiv_rn(red[0], 127.0f) : 1.0f;
    if (threadIdx.x == 0) s_w[o] = s;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        float t = rintf(__fdiv_rn(row[k], s));
        t = fminf(fmaxf(t, -127.f), 127.f);
        q[(long long)o * K + k] = (int8_t)t;
    }
}

// max |x| of the real-valued input: frames are u / 255, vectors are taken as they are
__global__ void input_absmax_kernel(const void *obs, long long n, int is_u8, float *out)
{
    float m = 0.f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        m = fmaxf(m, is_u8 ? __fdiv_rn((float)((const uint8_t *)obs)[i], 255.0f) : fabsf(((const float *)obs)[i]));
    if (m > 0.f) atomic_max_nonneg(out, m);
}

__global__ void input_quantise_kernel(const void *obs, long long n, int is_u8, float s_input, int8_t *q)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float x = is_u8 ? __fdiv_rn((float)((const uint8_t *)obs)[i], 255.0f) : ((const float *)obs)[i];
    float t = rintf(__fdiv_rn(x, s_input));
    t = fminf(fmaxf(t, -128.f), 127.f);
    q[i] = (int8_t)t;
}

struct CalibLayer {
    int in_c, in_h, in_w, out_c, out_h, out_w, kh, kw, stride, pad, relu_in, relu_out;
};

// int32 accumulators of a conv or fc layer (fc: 1 x 1 spatial), NCHW int8 in, residual added
__global__ void calib_acc_kernel(const int8_t *x, const int8_t *w, const int8_t *skip, const int *skip_mul,
                                 CalibLayer L, long long total, int *acc)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int ox = (int)(idx % L.out_w);
    long long t = idx / L.out_w;
    const int oy = (int)(t % L.out_h);
    t /= L.out_h;
    const int oc = (int)(t % L.out_c);
    const long long n = t / L.out_c;
    int a = 0;
    for (int c = 0; c < L.in_c; ++c)
        for (int ky = 0; ky < L.kh; ++ky) {
            const int iy = oy * L.stride + ky - L.pad;
            if (iy < 0 || iy >= L.in_h) continue;
            for (int kx = 0; kx < L.kw; ++kx) {
                const int ix = ox * L.stride + kx - L.pad;
                if (ix < 0 || ix >= L.in_w) continue;
                int xv = x[((n * L.in_c + c) * L.in_h + iy) * L.in_w + ix];
                if (L.relu_in && xv < 0) xv = 0;
                a += xv * (int)w[((oc * L.in_c + c) * L.kh + ky) * L.kw + kx];
            }
        }
    if (skip) a += skip_mul[oc] * (int)skip[idx];
    acc[idx] = a;
}

// y = fmaf((float)acc, s_in * s_w[c], b[c]) (+ ReLU); pass 0: max|y| into *ymax, pass 1: requantise
__global__ void calib_epilogue_kernel(const int *acc, const float *kscale, const float *bias, CalibLayer L,
                                      long long total, int pass, float s_out, float *ymax, int8_t *q)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int oc = (int)((idx / ((long long)L.out_h * L.out_w)) % L.out_c);
    float y = __fmaf_rn(__int2float_rn(acc[idx]), kscale[oc], bias[oc]);
    if (L.relu_out) y = fmaxf(y, 0.f);
    if (pass == 0) {
        const float a = fabsf(y);
        if (a > 0.f) atomic_max_nonneg(ymax, a);
    } else {
        float t = rintf(__fdiv_rn(y, s_out));
        t = fminf(fmaxf(t, -128.f), 127.f);
        q[idx] = (int8_t)t;
    }
}

__global__ void calib_maxpool_kernel(const int8_t *x, CalibLayer L, long long total, int8_t *q)
{
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int ox = (int)(idx % L.out_w);
    long long t = idx / L.out_w;
    const int oy = (int)(t % L.out_h);
    t /= L.out_h;  // t = n * C + c
    int m = -128;
    for (int ky = 0; ky < L.kh; ++ky)
        for (int kx = 0; kx < L.kw; ++kx)
            m = max(m, (int)x[(t * L.in_h + oy * L.stride + ky) * L.in_w + ox * L.stride + kx]);
    q[idx] = (int8_t)m;
}

struct DevMem {  // frees what it holds
    std::vector<void *> ptrs;
    ~DevMem()
    {
        for (void *p : ptrs) cudaFree(p);
    }
    template <typename T>
    cudaError_t get(T **out, size_t count)
    {
        void *d = nullptr;
        cudaError_t e = cudaMalloc(&d, count * sizeof(T) + 16);
        if (e == cudaSuccess) ptrs.push_back(d);
        *out = (T *)d;
        return e;
    }
};

unsigned blocks_for(long long n) { return (unsigned)((n + 255) / 256); }

}  // namespace

}  // namespace accerl

using namespace accerl;

extern "C" accerl_status accerl_policy_create_fp32(accerl_policy **out, int32_t in_kind,
                                                   const int32_t in_shape[3],
                                                   const accerl_layer_fp32 *layers, int32_t n_layers,
                                                   const void *calib_obs_host, int32_t calib_rows,
                                                   int32_t prune_2_4, int32_t max_batch, uint32_t flags,
                                                   int32_t device)
{
    if (out) *out = nullptr;
    if (!out || !in_shape || !layers || !calib_obs_host) {
        set_error("create_fp32: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if ((in_kind != ACCERL_IN_U8_NCHW && in_kind != ACCERL_IN_F32) || n_layers < 1 || n_layers > 4096 ||
        calib_rows < 1 || calib_rows > (1 << 20) || in_shape[0] < 1 || in_shape[1] < 1 || in_shape[2] < 1) {
        set_error("create_fp32: bad input kind, shape, layer count or calibration rows");
        return ACCERL_ERR_INVALID_ARG;
    }
    // shapes (the full validation is accerl_policy_create's; here only what the kernels index with)
    struct Shape {
        int c, h, w;
    };
    std::vector<Shape> shapes;
    Shape cur{in_shape[0], in_shape[1], in_shape[2]};
    size_t max_elems = (size_t)cur.c * cur.h * cur.w;
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_fp32 &d = layers[i];
        Shape o;
        if (d.kind == ACCERL_FC) {
            if ((long long)cur.c * cur.h * cur.w != d.in_c || d.out_c < 1) {
                set_error("create_fp32: layer %d: FC expects in_c = %lld", i, (long long)cur.c * cur.h * cur.w);
                return ACCERL_ERR_INVALID_ARG;
            }
            o = Shape{d.out_c, 1, 1};
        } else if (d.kind == ACCERL_CONV2D || d.kind == ACCERL_MAXPOOL) {
            if (d.in_c != cur.c || d.in_h != cur.h || d.in_w != cur.w || d.kh < 1 || d.kw != d.kh || d.stride < 1 ||
                d.pad < 0 || d.pad >= d.kh || d.out_c < 1 || cur.h + 2 * d.pad < d.kh || cur.w + 2 * d.pad < d.kw ||
                (d.kind == ACCERL_MAXPOOL && (d.pad != 0 || d.out_c != d.in_c))) {
                set_error("create_fp32: layer %d: shape does not follow from the previous layer", i);
                return ACCERL_ERR_INVALID_ARG;
            }
            o = Shape{d.out_c, (cur.h + 2 * d.pad - d.kh) / d.stride + 1, (cur.w + 2 * d.pad - d.kw) / d.stride + 1};
        } else {
            set_error("create_fp32: layer %d: unknown kind %d", i, d.kind);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (d.kind != ACCERL_MAXPOOL && (!d.w || !d.bias)) {
            set_error("create_fp32: layer %d: w and bias must be non-null", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (d.skip_from >= i || d.skip_from < -1 ||
            (d.skip_from >= 0 && (d.kind != ACCERL_CONV2D || shapes[d.skip_from].c != o.c ||
                                  shapes[d.skip_from].h != o.h || shapes[d.skip_from].w != o.w))) {
            set_error("create_fp32: layer %d: skip_from must name an earlier layer with this layer's output shape", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (prune_2_4 && d.kind != ACCERL_MAXPOOL && ((long long)d.in_c * d.kh * d.kw) % 4) {
            set_error("create_fp32: layer %d: 2:4 pruning needs K to be a multiple of 4", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        shapes.push_back(o);
        max_elems = std::max(max_elems, (size_t)o.c * o.h * o.w);
        cur = o;
    }
    if (max_elems * (size_t)calib_rows >= ((size_t)1 << 33)) {
        set_error("create_fp32: calibration batch too large (%zu elements per tensor)", max_elems * (size_t)calib_rows);
        return ACCERL_ERR_UNSUPPORTED;
    }
    int ndev = 0, prev = -1;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        set_error("create_fp32: CUDA device %d not available", device);
        cudaGetLastError();
        return ACCERL_ERR_CUDA;
    }
    cudaGetDevice(&prev);
    struct Restore {
        int prev;
        ~Restore() { if (prev >= 0) cudaSetDevice(prev); }
    } restore{prev};
    ACCERL_CUDA_TRY(cudaSetDevice(device));

    const long long B = calib_rows;
    const long long in_elems = (long long)in_shape[0] * in_shape[1] * in_shape[2] * B;
    const bool u8 = in_kind == ACCERL_IN_U8_NCHW;
    DevMem mem;
    // ---- input scale and quantised calibration batch
    void *obs_dev = nullptr;
    ACCERL_CUDA_TRY(mem.get((uint8_t **)&obs_dev, (size_t)in_elems * (u8 ? 1 : 4)));
    ACCERL_CUDA_TRY(cudaMemcpy(obs_dev, calib_obs_host, (size_t)in_elems * (u8 ? 1 : 4), cudaMemcpyHostToDevice));
    float *scal = nullptr;  // [0]: running maximum
    ACCERL_CUDA_TRY(mem.get(&scal, 4));
    ACCERL_CUDA_TRY(cudaMemset(scal, 0, 16));
    input_absmax_kernel<<<1024, 256>>>(obs_dev, in_elems, u8 ? 1 : 0, scal);
    float m = 0.f;
    ACCERL_CUDA_TRY(cudaMemcpy(&m, scal, 4, cudaMemcpyDeviceToHost));
    volatile float s_input_v = m > 0.f ? m / 127.0f : 1.0f;
    const float s_input = s_input_v;
    std::vector<int8_t *> act(n_layers + 1, nullptr);  // act[t + 1]: int8 NCHW tensor t of the calibration batch
    ACCERL_CUDA_TRY(mem.get(&act[0], (size_t)in_elems));
    input_quantise_kernel<<<blocks_for(in_elems), 256>>>(obs_dev, in_elems, u8 ? 1 : 0, s_input, act[0]);
    ACCERL_CUDA_TRY(cudaGetLastError());
    int *acc = nullptr;
    ACCERL_CUDA_TRY(mem.get(&acc, max_elems * (size_t)B));

    // ---- layer by layer
    struct Quant {
        std::vector<int8_t> w;
        std::vector<float> s_w, bias;
        std::vector<int32_t> skip_mul;
        float s_in = 1.f, s_out = 1.f;
    };
    std::vector<Quant> Q;
    try {
        Q.resize(n_layers);
    } catch (const std::bad_alloc &) {
        set_error("create_fp32: out of host memory");
        return ACCERL_ERR_OOM;
    }
    std::vector<float> scales(n_layers, 1.f);
    float s_prev = s_input;
    Shape in{in_shape[0], in_shape[1], in_shape[2]};
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_fp32 &d = layers[i];
        const Shape o = shapes[i];
        const long long out_elems = (long long)o.c * o.h * o.w * B;
        CalibLayer L{in.c, in.h, in.w, o.c, o.h, o.w, d.kh, d.kw, d.stride, d.pad,
                     (d.flags & ACCERL_RELU_IN) ? 1 : 0, (d.flags & ACCERL_RELU_OUT) ? 1 : 0};
        Quant &q = Q[i];
        q.s_in = s_prev;
        const bool last = (d.flags & ACCERL_LOGITS) != 0;
        if (d.kind == ACCERL_MAXPOOL) {
            ACCERL_CUDA_TRY(mem.get(&act[i + 1], (size_t)out_elems));
            calib_maxpool_kernel<<<blocks_for(out_elems), 256>>>(act[i], L, out_elems, act[i + 1]);
            ACCERL_CUDA_TRY(cudaGetLastError());
            q.s_out = s_prev;
        } else {
            if (d.kind == ACCERL_FC) {
                L.in_c = d.in_c;
                L.in_h = L.in_w = L.kh = L.kw = L.stride = 1;
                L.pad = 0;
            }
            const int K = L.in_c * L.kh * L.kw;
            const size_t nw = (size_t)o.c * K;
            float *w_dev = nullptr, *sw_dev = nullptr, *k_dev = nullptr, *b_dev = nullptr;
            int8_t *wq_dev = nullptr;
            ACCERL_CUDA_TRY(mem.get(&w_dev, nw));
            ACCERL_CUDA_TRY(mem.get(&sw_dev, (size_t)o.c));
            ACCERL_CUDA_TRY(mem.get(&k_dev, (size_t)o.c));
            ACCERL_CUDA_TRY(mem.get(&b_dev, (size_t)o.c));
            ACCERL_CUDA_TRY(mem.get(&wq_dev, nw));
            ACCERL_CUDA_TRY(cudaMemcpy(w_dev, d.w, nw * 4, cudaMemcpyHostToDevice));
            ACCERL_CUDA_TRY(cudaMemcpy(b_dev, d.bias, (size_t)o.c * 4, cudaMemcpyHostToDevice));
            if (prune_2_4) prune24_kernel<<<blocks_for((long long)nw / 4), 256>>>(w_dev, o.c, L.in_c, L.kh, L.kw);
            quantise_weights_kernel<<<(unsigned)o.c, 256>>>(w_dev, K, sw_dev, wq_dev);
            ACCERL_CUDA_TRY(cudaGetLastError());
            q.w.resize(nw);
            q.s_w.resize(o.c);
            q.bias.assign(d.bias, d.bias + o.c);
            ACCERL_CUDA_TRY(cudaMemcpy(q.w.data(), wq_dev, nw, cudaMemcpyDeviceToHost));
            ACCERL_CUDA_TRY(cudaMemcpy(q.s_w.data(), sw_dev, (size_t)o.c * 4, cudaMemcpyDeviceToHost));
            std::vector<float> ks(o.c);
            for (int c = 0; c < o.c; ++c) {
                volatile float k = s_prev * q.s_w[c];  // one fp32 rounding
                ks[c] = k;
            }
            ACCERL_CUDA_TRY(cudaMemcpy(k_dev, ks.data(), (size_t)o.c * 4, cudaMemcpyHostToDevice));
            int *sm_dev = nullptr;
            if (d.skip_from >= 0) {
                // integer multiplier that brings the skip tensor (scale s_x) onto the accumulators' grid
                q.skip_mul.resize(o.c);
                const float s_x = scales[d.skip_from];
                for (int c = 0; c < o.c; ++c) {
                    volatile float r = s_x / ks[c];
                    float rr = rintf(r);
                    rr = rr < 0.f ? 0.f : (rr > 32767.f ? 32767.f : rr);
                    q.skip_mul[c] = (int32_t)rr;
                }
                ACCERL_CUDA_TRY(mem.get(&sm_dev, (size_t)o.c));
                ACCERL_CUDA_TRY(cudaMemcpy(sm_dev, q.skip_mul.data(), (size_t)o.c * 4, cudaMemcpyHostToDevice));
            }
            calib_acc_kernel<<<blocks_for(out_elems), 256>>>(act[i], wq_dev, d.skip_from >= 0 ? act[d.skip_from + 1] : nullptr,
                                                             sm_dev, L, out_elems, acc);
            ACCERL_CUDA_TRY(cudaGetLastError());
            q.s_out = 1.0f;
            if (!last) {
                ACCERL_CUDA_TRY(cudaMemset(scal, 0, 4));
                calib_epilogue_kernel<<<blocks_for(out_elems), 256>>>(acc, k_dev, b_dev, L, out_elems, 0, 1.f, scal, nullptr);
                float ym = 0.f;
                ACCERL_CUDA_TRY(cudaMemcpy(&ym, scal, 4, cudaMemcpyDeviceToHost));
                volatile float so = ym > 0.f ? ym / 127.0f : 1.0f;
                q.s_out = so;
                ACCERL_CUDA_TRY(mem.get(&act[i + 1], (size_t)out_elems));
                calib_epilogue_kernel<<<blocks_for(out_elems), 256>>>(acc, k_dev, b_dev, L, out_elems, 1, q.s_out, scal,
                                                                      act[i + 1]);
                ACCERL_CUDA_TRY(cudaGetLastError());
            }
        }
        scales[i] = q.s_out;
        s_prev = q.s_out;
        in = o;
        if (last) break;
    }
    ACCERL_CUDA_TRY(cudaDeviceSynchronize());

    // ---- hand the quantised network to the ordinary constructor
    std::vector<accerl_layer_desc> descs(n_layers);
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_fp32 &d = layers[i];
        accerl_layer_desc &e = descs[i];
        memset(&e, 0, sizeof(e));
        e.kind = d.kind;
        e.flags = d.flags;
        e.in_c = d.in_c; e.in_h = d.in_h; e.in_w = d.in_w; e.out_c = d.out_c;
        e.kh = d.kh; e.kw = d.kw; e.stride = d.stride; e.pad = d.pad;
        e.s_in = Q[i].s_in;
        e.s_out = Q[i].s_out;
        e.skip_from = d.skip_from;
        if (d.kind != ACCERL_MAXPOOL) {
            e.w = Q[i].w.data();
            e.s_w = Q[i].s_w.data();
            e.bias = Q[i].bias.data();
            e.skip_mul = d.skip_from >= 0 ? Q[i].skip_mul.data() : nullptr;
        }
    }
    accerl_status st = accerl_policy_create(out, in_kind, in_shape, s_input, descs.data(), n_layers, max_batch,
                                            flags, device);
    if (st != ACCERL_OK) return st;
    // keep the quantised parameters for accerl_policy_export
    accerl_policy *p = *out;
    p->ptq.resize(n_layers);
    for (int i = 0; i < n_layers; ++i) {
        p->ptq[i].w = std::move(Q[i].w);
        p->ptq[i].s_w = std::move(Q[i].s_w);
        p->ptq[i].skip_mul = std::move(Q[i].skip_mul);
        p->ptq[i].s_in = Q[i].s_in;
        p->ptq[i].s_out = Q[i].s_out;
    }
    return ACCERL_OK;
}

extern "C" accerl_status accerl_policy_export(const accerl_policy *p, int32_t layer, int8_t *w_host,
                                              size_t w_bytes, float *s_w_host, int32_t *skip_mul_host,
                                              float *s_in_out, float *s_out_out)
{
    if (!p) {
        set_error("export: null handle");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (p->ptq.empty()) {
        set_error("export: the handle was not built by accerl_policy_create_fp32");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (layer < 0 || layer >= (int)p->ptq.size()) {
        set_error("export: layer %d out of range", layer);
        return ACCERL_ERR_INVALID_ARG;
    }
    const accerl_policy::PtqLayer &q = p->ptq[layer];
    if (s_in_out) *s_in_out = q.s_in;
    if (s_out_out) *s_out_out = q.s_out;
    if (w_host) {
        if (w_bytes < q.w.size()) {
            set_error("export: w_host holds %zu bytes, %zu needed", w_bytes, q.w.size());
            return ACCERL_ERR_INVALID_ARG;
        }
        if (!q.w.empty()) memcpy(w_host, q.w.data(), q.w.size());
    }
    if (s_w_host && !q.s_w.empty()) memcpy(s_w_host, q.s_w.data(), q.s_w.size() * sizeof(float));
    if (skip_mul_host && !q.skip_mul.empty()) memcpy(skip_mul_host, q.skip_mul.data(), q.skip_mul.size() * sizeof(int32_t));
    return ACCERL_OK;
}
