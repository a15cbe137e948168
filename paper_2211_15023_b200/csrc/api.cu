// Host side of the library: validation, weight repacking, workspace planning and the launch
// sequence behind the extern "C" entry points declared in accerl.h.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "internal.h"

namespace accerl {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

template <typename T>
accerl_status upload(accerl_policy *p, const std::vector<T> &host, T **dev)
{
    *dev = nullptr;
    size_t bytes = std::max<size_t>(host.size() * sizeof(T), 16);
    void *d = nullptr;
    ACCERL_CUDA_TRY(cudaMalloc(&d, bytes));
    p->owned.push_back(d);
    if (!host.empty())
        ACCERL_CUDA_TRY(cudaMemcpy(d, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice));
    *dev = (T *)d;
    return ACCERL_OK;
}

struct Shape {
    int c, h, w;
};

bool good_scale(float s) { return s > 0.f && isfinite(s); }

// Checks one descriptor against the tensor it consumes; fills the shape it produces.
accerl_status validate_layer(const accerl_layer_desc &d, int i, int n_layers, Shape in, float s_run,
                             const std::vector<Shape> &outs, Shape *out)
{
    const bool last = i == n_layers - 1;
    if (d.kind != ACCERL_CONV2D && d.kind != ACCERL_FC && d.kind != ACCERL_MAXPOOL) {
        set_error("layer %d: unknown kind %d", i, d.kind);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (d.flags & ~(uint32_t)(ACCERL_RELU_IN | ACCERL_RELU_OUT | ACCERL_LOGITS)) {
        set_error("layer %d: unknown flag bits 0x%x", i, d.flags);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (((d.flags & ACCERL_LOGITS) != 0) != last || (last && d.kind != ACCERL_FC)) {
        set_error("layer %d: the last layer, and only it, must be an FC with ACCERL_LOGITS", i);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (!good_scale(d.s_in) || !good_scale(d.s_out)) {
        set_error("layer %d: scales must be positive and finite", i);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (d.s_in != s_run) {
        set_error("layer %d: s_in %.9g differs from the scale of the tensor it reads (%.9g)", i,
                  d.s_in, s_run);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (d.in_c < 1 || d.out_c < 1 || d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0) {
        set_error("layer %d: non-positive size", i);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (d.kind == ACCERL_FC) {
        if ((long long)in.c * in.h * in.w != d.in_c || d.kh != 1 || d.kw != 1 || d.stride != 1 ||
            d.pad != 0 || d.in_h != 1 || d.in_w != 1) {
            set_error("layer %d: FC expects in_c = %lld (flattened input) and unit kernel fields", i,
                      (long long)in.c * in.h * in.w);
            return ACCERL_ERR_INVALID_ARG;
        }
        *out = Shape{d.out_c, 1, 1};
    } else {
        if (d.in_c != in.c || d.in_h != in.h || d.in_w != in.w) {
            set_error("layer %d: input %dx%dx%d does not match the previous output %dx%dx%d", i,
                      d.in_c, d.in_h, d.in_w, in.c, in.h, in.w);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (d.kh != d.kw) {
            set_error("layer %d: only square windows are supported", i);
            return ACCERL_ERR_UNSUPPORTED;
        }
        int oh = (d.in_h + 2 * d.pad - d.kh) / d.stride + 1;
        int ow = (d.in_w + 2 * d.pad - d.kw) / d.stride + 1;
        if (d.in_h + 2 * d.pad < d.kh || d.in_w + 2 * d.pad < d.kw || oh < 1 || ow < 1) {
            set_error("layer %d: window larger than the padded input", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (d.kind == ACCERL_MAXPOOL && (d.out_c != d.in_c || d.pad != 0 || d.s_out != d.s_in ||
                                         d.flags != 0 || d.skip_from >= 0)) {
            set_error("layer %d: max-pool needs out_c = in_c, pad 0, s_out = s_in, no flags", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        if (d.pad >= d.kh) {
            set_error("layer %d: pad must be smaller than the window", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        *out = Shape{d.out_c, oh, ow};
    }
    if (d.kind != ACCERL_MAXPOOL) {
        if (!d.w || !d.s_w || !d.bias) {
            set_error("layer %d: w, s_w and bias must be non-null", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        long long k = (long long)d.in_c * d.kh * d.kw;
        if (k * 127 * 128 + 32767LL * 128 >= 2147483647LL) {
            set_error("layer %d: K = %lld could overflow the int32 accumulator", i, k);
            return ACCERL_ERR_UNSUPPORTED;
        }
        long long nw = k * d.out_c;
        for (long long j = 0; j < nw; ++j)
            if (d.w[j] == -128) {
                set_error("layer %d: weight %lld is -128 (symmetric int8 uses [-127, 127])", i, j);
                return ACCERL_ERR_INVALID_ARG;
            }
        for (int c = 0; c < d.out_c; ++c)
            if (!good_scale(d.s_w[c]) || !isfinite(d.bias[c])) {
                set_error("layer %d: s_w[%d] / bias[%d] not usable", i, c, c);
                return ACCERL_ERR_INVALID_ARG;
            }
    }
    if (d.skip_from >= 0) {
        if (d.kind != ACCERL_CONV2D) {
            set_error("layer %d: residual add is supported on conv layers only", i);
            return ACCERL_ERR_UNSUPPORTED;
        }
        if (d.skip_from >= i || !d.skip_mul) {
            set_error("layer %d: skip_from must name an earlier layer and skip_mul be non-null", i);
            return ACCERL_ERR_INVALID_ARG;
        }
        Shape s = outs[d.skip_from];
        if (s.c != out->c || s.h != out->h || s.w != out->w) {
            set_error("layer %d: skip tensor %dx%dx%d differs from the output %dx%dx%d", i, s.c, s.h,
                      s.w, out->c, out->h, out->w);
            return ACCERL_ERR_INVALID_ARG;
        }
        for (int c = 0; c < d.out_c; ++c)
            if (d.skip_mul[c] < 0 || d.skip_mul[c] > 32767) {
                set_error("layer %d: skip_mul[%d] outside [0, 32767]", i, c);
                return ACCERL_ERR_INVALID_ARG;
            }
    } else if (d.skip_from != -1 || d.skip_mul) {
        set_error("layer %d: skip_from must be -1 with a null skip_mul, or a layer index", i);
        return ACCERL_ERR_INVALID_ARG;
    }
    return ACCERL_OK;
}

// Repack OIHW int8 weights into the word layouts of the generic kernels.
void pack_generic(const accerl_layer_desc &d, LayerPlan &L, std::vector<int32_t> &words)
{
    const int C4 = L.in_cp / 4;
    if (d.kind == ACCERL_CONV2D) {
        words.assign((size_t)d.kh * d.kw * C4 * L.oc_pad, 0);
        for (int oc = 0; oc < d.out_c; ++oc)
            for (int ic = 0; ic < d.in_c; ++ic)
                for (int ky = 0; ky < d.kh; ++ky)
                    for (int kx = 0; kx < d.kw; ++kx) {
                        int8_t v = d.w[((oc * d.in_c + ic) * d.kh + ky) * d.kw + kx];
                        size_t wi = ((size_t)(ky * d.kw + kx) * C4 + ic / 4) * L.oc_pad + oc;
                        words[wi] |= (int32_t)((uint32_t)(uint8_t)v << (8 * (ic % 4)));
                    }
    } else {
        // FC input is the previous tensor in (y, x, c) order with c padded to in_cp; the
        // descriptor's columns are in (c, y, x) order
        const int K_int = L.in_h * L.in_w * L.in_cp;
        words.assign((size_t)L.oc_pad * (K_int / 4), 0);
        for (int oc = 0; oc < d.out_c; ++oc)
            for (int c = 0; c < L.in_c; ++c)
                for (int y = 0; y < L.in_h; ++y)
                    for (int x = 0; x < L.in_w; ++x) {
                        int8_t v = d.w[(size_t)oc * d.in_c + (c * L.in_h + y) * L.in_w + x];
                        int ki = (y * L.in_w + x) * L.in_cp + c;
                        words[(size_t)oc * (K_int / 4) + ki / 4] |=
                            (int32_t)((uint32_t)(uint8_t)v << (8 * (ki % 4)));
                    }
    }
}

}  // namespace

accerl_status upload_bytes(accerl_policy *p, const void *host, size_t bytes, void **dev)
{
    *dev = nullptr;
    void *d = nullptr;
    ACCERL_CUDA_TRY(cudaMalloc(&d, bytes < 16 ? 16 : bytes));
    p->owned.push_back(d);
    ACCERL_CUDA_TRY(cudaMemcpy(d, host, bytes, cudaMemcpyHostToDevice));
    *dev = d;
    return ACCERL_OK;
}

}  // namespace accerl

using namespace accerl;

// argument checks shared by the act entry points (nothing is launched when they fail)
static accerl_status check_act_args(accerl_policy *p, const void *obs_dev,
                                    const float *uniforms_dev, int32_t batch, float *logits_dev,
                                    int32_t *actions_dev, float *logp_dev)
{
    if (!p || !obs_dev || !uniforms_dev || !logits_dev || !actions_dev || !logp_dev) {
        set_error("act: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch < 1) {
        set_error("act: batch must be at least 1");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch > p->max_batch) {
        set_error("act: batch %d exceeds max_batch %d", batch, p->max_batch);
        return ACCERL_ERR_BATCH_TOO_LARGE;
    }
    if (((uintptr_t)obs_dev & 15) || ((uintptr_t)uniforms_dev & 3) || ((uintptr_t)logits_dev & 3) ||
        ((uintptr_t)actions_dev & 3) || ((uintptr_t)logp_dev & 3)) {
        set_error("act: misaligned pointer (obs needs 16 bytes, the others 4)");
        return ACCERL_ERR_INVALID_ARG;
    }
    return ACCERL_OK;
}

// Enqueue the plan's launches; with `ev`, record ev[i] before launch i and ev[n] after the last.
static accerl_status run_steps(accerl_policy *p, const void *obs_dev, const float *uniforms_dev,
                               int B, float *logits_dev, int32_t *actions_dev, float *logp_dev,
                               float *value_dev, float *entropy_dev, cudaStream_t st, cudaEvent_t *ev)
{
    p->last_stream = st;
    // a last layer with a value column and a sampler launch of its own: the layer's floats go to
    // the handle's scratch rows of n_out, the sampler splits them into logits and value
    float *z_dev = p->n_out != p->n_actions ? p->z_scratch : logits_dev;
    for (size_t i = 0; i < p->steps.size(); ++i) {
        const Step &s = p->steps[i];
        if (ev) ACCERL_CUDA_TRY(cudaEventRecord(ev[i], st));
        const LayerPlan *L = s.layer >= 0 ? &p->layers[s.layer] : nullptr;
        const int8_t *in = L ? p->bufs[L->in_buf].ptr : nullptr;
        int8_t *o = L && L->out_buf >= 0 ? p->bufs[L->out_buf].ptr : nullptr;
        switch (s.kind) {
        case Step::INGEST: {
            int8_t *x = p->bufs[p->layers[0].in_buf].ptr;
            if (p->in_kind == ACCERL_IN_U8_NCHW)
                ACCERL_CUDA_TRY(launch_ingest_u8((const uint8_t *)obs_dev, p->lut, x, B, p->in_c,
                                                 p->in_h, p->in_w, p->in_cp, st));
            else
                ACCERL_CUDA_TRY(launch_ingest_f32((const float *)obs_dev, p->s_input, x, B, p->in_c,
                                                  p->in_cp, st));
            break;
        }
        case Step::CONV_GENERIC:
            ACCERL_CUDA_TRY(launch_conv_generic(
                *L, in, L->skip_buf >= 0 ? p->bufs[L->skip_buf].ptr : nullptr, o, B, st));
            break;
        case Step::FC_GENERIC:
            ACCERL_CUDA_TRY(launch_fc_generic(*L, in, o, z_dev, B, st));
            break;
        case Step::POOL_GENERIC:
            ACCERL_CUDA_TRY(launch_maxpool_generic(*L, in, o, B, st));
            break;
        case Step::INGEST_S2D:
            ACCERL_CUDA_TRY(launch_ingest_u8_s2d((const uint8_t *)obs_dev, p->lut,
                                                 p->bufs[p->layers[0].in_buf].ptr, B, p->in_c,
                                                 p->in_h, p->in_w, p->tensor_s2d[0], p->ingest_arith,
                                                 p->ingest_mul, p->ingest_add, st));
            break;
        case Step::TC_GEMM: {
            TcStep &t = p->tc_steps[s.tc];
            TcGemmParams prm = t.prm;
            prm.batch = B;
            prm.m_tiles = (int)(((long long)B * prm.rows_per_image + 127) / 128);
            prm.logits = prm.logits_mode ? z_dev : nullptr;
            if (prm.fuse_ingest) {
                if ((uintptr_t)obs_dev & 15) {
                    set_error("act: this plan reads the frames with 16-byte bulk copies; obs_dev must be 16-byte aligned");
                    return ACCERL_ERR_INVALID_ARG;
                }
                prm.obs = (const uint8_t *)obs_dev;
            }
            ACCERL_CUDA_TRY(tc_launch(t.map_a, t.map_b, prm, t.resident_b, p->sm_count, st));
            break;
        }
        case Step::CONV1_FRAMES:
            if ((uintptr_t)obs_dev & 15) {
                set_error("act: obs_dev must be 16-byte aligned");
                return ACCERL_ERR_INVALID_ARG;
            }
            ACCERL_CUDA_TRY(conv1_launch(p->conv1_map_b, p->conv1, B, (const uint8_t *)obs_dev, p->sm_count, st));
            break;
        case Step::CONV_ROWS: {
            const ConvRowsStep &cs = p->conv_rows[s.tc];
            ACCERL_CUDA_TRY(conv_rows_launch(cs.map_a, cs.map_b, cs.prm, B, p->sm_count, st));
            break;
        }
        case Step::INGEST_NHWC4:
            ACCERL_CUDA_TRY(launch_ingest_u8_nhwc4((const uint8_t *)obs_dev, p->lut,
                                                   p->bufs[p->layers[0].in_buf].ptr, B, p->in_h,
                                                   p->in_w, p->in_h, p->in_w, 0, 0,
                                                   p->ingest_shift1 ? 4 : (p->ingest_float ? 2 : p->ingest_arith),
                                                   p->ingest_float ? p->ingest_fa : p->ingest_mul,
                                                   p->ingest_float ? p->ingest_fc1 : p->ingest_add, st));
            break;
        case Step::INGEST_PAD4:
            ACCERL_CUDA_TRY(launch_ingest_u8_nhwc4((const uint8_t *)obs_dev, p->lut, p->in_pad4, B,
                                                   p->in_h, p->in_w, p->in_h + 2, p->in_pad4_w, 1, 4,
                                                   p->ingest_shift1 ? 4 : (p->ingest_float ? 2 : p->ingest_arith),
                                                   p->ingest_float ? p->ingest_fa : p->ingest_mul,
                                                   p->ingest_float ? p->ingest_fc1 : p->ingest_add, st));
            break;
        case Step::POOL_DUAL:
            ACCERL_CUDA_TRY(launch_maxpool_dual(p->pools[s.tc], B, st));
            break;
        case Step::MLP_FUSED:
            ACCERL_CUDA_TRY(launch_mlp_fused(p, (const float *)obs_dev, uniforms_dev, B, logits_dev,
                                             actions_dev, logp_dev, value_dev, entropy_dev, st));
            break;
        case Step::FC_SAMPLE:
            ACCERL_CUDA_TRY(launch_fc_sample(p->fc_sample, uniforms_dev, B, logits_dev, actions_dev, logp_dev,
                                             value_dev, entropy_dev, p->sm_count, st));
            break;
        case Step::SAMPLE:
            ACCERL_CUDA_TRY(launch_sample(z_dev, p->n_out, uniforms_dev, B, p->n_actions,
                                          z_dev != logits_dev ? logits_dev : nullptr, actions_dev,
                                          logp_dev, value_dev, entropy_dev, st));
            break;
        }
    }
    if (ev) ACCERL_CUDA_TRY(cudaEventRecord(ev[p->steps.size()], st));
    return ACCERL_OK;
}

extern "C" {

const char *accerl_last_error(void) { return g_err; }
const char *accerl_version(void) { return "accerl-b200 0.1 (sm_100a)"; }

void accerl_policy_destroy(accerl_policy *p)
{
    if (!p) return;
    DeviceGuard g(p->device);
    cudaDeviceSynchronize();
    for (void *d : p->owned) cudaFree(d);
    for (cudaEvent_t ev : p->events) cudaEventDestroy(ev);
    for (cudaEvent_t ev : p->copy_events) cudaEventDestroy(ev);
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    delete p;
}

accerl_status accerl_policy_create(accerl_policy **out, int32_t in_kind, const int32_t in_shape[3],
                                   float s_input, const accerl_layer_desc *layers,
                                   int32_t n_layers, int32_t max_batch, uint32_t flags,
                                   int32_t device)
{
    if (out) *out = nullptr;
    if (!out || !in_shape || !layers) {
        set_error("create: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (in_kind != ACCERL_IN_U8_NCHW && in_kind != ACCERL_IN_F32) {
        set_error("create: unknown input kind %d", in_kind);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (in_shape[0] < 1 || in_shape[1] < 1 || in_shape[2] < 1 ||
        (in_kind == ACCERL_IN_F32 && (in_shape[1] != 1 || in_shape[2] != 1))) {
        set_error("create: bad input shape");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (n_layers < 1 || n_layers > 4096 || max_batch < 1 || !good_scale(s_input)) {
        set_error("create: n_layers, max_batch and s_input must be positive");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (flags & ~(uint32_t)(ACCERL_FLAG_KEEP_ACTIVATIONS | ACCERL_FLAG_FORCE_GENERIC | ACCERL_FLAG_TAP_FUSED |
                            ACCERL_FLAG_VALUE_HEAD | ACCERL_FLAG_TEST_NO_FASTDIV |
                            ACCERL_FLAG_TEST_NO_AFFINE)) {
        set_error("create: unknown flag bits 0x%x", flags);
        return ACCERL_ERR_INVALID_ARG;
    }
    if ((flags & ACCERL_FLAG_TAP_FUSED) && !(flags & ACCERL_FLAG_KEEP_ACTIVATIONS)) {
        set_error("create: ACCERL_FLAG_TAP_FUSED needs ACCERL_FLAG_KEEP_ACTIVATIONS");
        return ACCERL_ERR_INVALID_ARG;
    }
    // ---- validate the chain on the host before touching the device
    std::vector<Shape> shapes;
    Shape cur{in_shape[0], in_shape[1], in_shape[2]};
    float s_run = s_input;
    for (int i = 0; i < n_layers; ++i) {
        Shape o;
        accerl_status st = validate_layer(layers[i], i, n_layers, cur, s_run, shapes, &o);
        if (st != ACCERL_OK) return st;
        shapes.push_back(o);
        cur = o;
        s_run = layers[i].s_out;
    }
    const bool value_head = (flags & ACCERL_FLAG_VALUE_HEAD) != 0;
    if (value_head && cur.c < 2) {
        set_error("create: ACCERL_FLAG_VALUE_HEAD needs a last layer with at least two columns (actions, then V)");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (cur.c - (value_head ? 1 : 0) > 1024) {
        set_error("create: %d actions (at most 1024 supported)", cur.c - (value_head ? 1 : 0));
        return ACCERL_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < n_layers; ++i) {
        long long px = (long long)max_batch * shapes[i].h * shapes[i].w;
        if (px * round_up(shapes[i].c, 4) >= (1LL << 40) || px >= (1LL << 31) * 128) {
            set_error("create: layer %d output too large for max_batch %d", i, max_batch);
            return ACCERL_ERR_UNSUPPORTED;
        }
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        set_error("create: CUDA device %d not available (%d devices)", device, ndev);
        cudaGetLastError();
        return ACCERL_ERR_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) {
        set_error("create: cudaSetDevice(%d) failed", device);
        return ACCERL_ERR_CUDA;
    }
    accerl_policy *p = new (std::nothrow) accerl_policy();
    if (!p) {
        set_error("create: out of host memory");
        return ACCERL_ERR_OOM;
    }
    p->device = device;
    p->in_kind = in_kind;
    p->in_c = in_shape[0];
    p->in_h = in_shape[1];
    p->in_w = in_shape[2];
    p->in_cp = round_up(p->in_c, 4);
    p->s_input = s_input;
    p->max_batch = max_batch;
    p->flags = flags;
    p->n_out = cur.c;
    p->n_actions = cur.c - (value_head ? 1 : 0);

    accerl_status st = ACCERL_OK;
    auto fail = [&](accerl_status s) {
        accerl_policy_destroy(p);
        return s;
    };

    // ---- layer plans and parameters
    Shape in{p->in_c, p->in_h, p->in_w};
    int in_cp = p->in_cp;
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        LayerPlan L;
        L.kind = d.kind;
        L.flags = d.flags;
        L.in_c = in.c; L.in_h = in.h; L.in_w = in.w; L.in_cp = in_cp;
        L.out_c = shapes[i].c; L.out_h = shapes[i].h; L.out_w = shapes[i].w;
        L.out_cp = round_up(L.out_c, 4);
        L.kh = d.kh; L.kw = d.kw; L.stride = d.stride; L.pad = d.pad;
        L.s_in = d.s_in; L.s_out = d.s_out;
        L.skip_from = d.skip_from;
        L.oc_pad = round_up(L.out_c, 16);
        if (d.kind != ACCERL_MAXPOOL) {
            std::vector<int32_t> words;
            pack_generic(d, L, words);
            std::vector<float> ks(L.oc_pad, 0.f), bs(L.oc_pad, 0.f);
            for (int c = 0; c < d.out_c; ++c) {
                volatile float k = d.s_in * d.s_w[c];  // one fp32 rounding, never contracted
                ks[c] = k;
                bs[c] = d.bias[c];
            }
            if ((st = upload(p, words, &L.w_generic)) != ACCERL_OK) return fail(st);
            if ((st = upload(p, ks, &L.kscale)) != ACCERL_OK) return fail(st);
            if ((st = upload(p, bs, &L.bias)) != ACCERL_OK) return fail(st);
            if (d.skip_from >= 0) {
                std::vector<int32_t> sm(L.oc_pad, 0);
                for (int c = 0; c < d.out_c; ++c) sm[c] = d.skip_mul[c];
                if ((st = upload(p, sm, &L.skip_mul)) != ACCERL_OK) return fail(st);
            }
            L.how = d.kind == ACCERL_CONV2D ? "conv_dp4a_kernel" : "fc_dp4a_kernel";
        } else {
            L.how = "maxpool_kernel";
        }
        p->layers.push_back(L);
        in = shapes[i];
        in_cp = L.out_cp;
    }

    // ---- workspace: tensor -1 is the quantised input, tensor i is layer i's int8 output.
    // Without KEEP_ACTIVATIONS a buffer is reused once its tensor has no reader left.
    const bool keep = (flags & ACCERL_FLAG_KEEP_ACTIVATIONS) != 0;
    std::vector<int> last_use(n_layers + 1, 0);  // indexed by tensor + 1
    for (int t = -1; t < n_layers - 1; ++t) last_use[t + 1] = t + 1;
    for (int i = 0; i < n_layers; ++i)
        if (layers[i].skip_from >= 0)
            last_use[layers[i].skip_from + 1] = std::max(last_use[layers[i].skip_from + 1], i);
    std::vector<int> buf_of(n_layers + 1, -1), free_after;  // free_after per physical buffer
    auto take = [&](size_t bytes, int producer, int until) {
        int best = -1;
        if (!keep)
            for (size_t b = 0; b < p->bufs.size(); ++b)
                if (free_after[b] < producer &&
                    (best < 0 || p->bufs[b].bytes_per_state > p->bufs[best].bytes_per_state))
                    best = (int)b;
        if (best < 0) {
            p->bufs.push_back(DeviceBuf());
            free_after.push_back(0);
            best = (int)p->bufs.size() - 1;
        }
        p->bufs[best].bytes_per_state = std::max(p->bufs[best].bytes_per_state, bytes);
        free_after[best] = until;
        return best;
    };
    buf_of[0] = take((size_t)p->in_h * p->in_w * p->in_cp, -1, last_use[0]);
    for (int i = 0; i < n_layers; ++i) {
        LayerPlan &L = p->layers[i];
        L.in_buf = buf_of[i];
        L.skip_buf = L.skip_from >= 0 ? buf_of[L.skip_from + 1] : -1;
        if (i < n_layers - 1) {
            buf_of[i + 1] = take((size_t)L.out_h * L.out_w * L.out_cp, i, last_use[i + 1]);
            L.out_buf = buf_of[i + 1];
        }
    }
    for (DeviceBuf &b : p->bufs) {
        size_t bytes = b.bytes_per_state * (size_t)max_batch + 256;
        void *d = nullptr;
        cudaError_t e = cudaMalloc(&d, bytes);
        if (e != cudaSuccess) {
            set_error("create: cudaMalloc of %zu workspace bytes failed: %s", bytes,
                      cudaGetErrorString(e));
            cudaGetLastError();
            return fail(e == cudaErrorMemoryAllocation ? ACCERL_ERR_OOM : ACCERL_ERR_CUDA);
        }
        p->owned.push_back(d);
        b.ptr = (int8_t *)d;
        p->workspace_bytes += bytes;
    }

    // ---- input table: the frame quantiser evaluated for all 256 byte values
    if (in_kind == ACCERL_IN_U8_NCHW) {
        std::vector<int8_t> lut(256);
        for (int u = 0; u < 256; ++u) {
            volatile float x = (float)u / 255.0f;
            volatile float t = x / s_input;
            float r = rintf(t);
            r = r < -128.f ? -128.f : (r > 127.f ? 127.f : r);
            lut[u] = (int8_t)r;
        }
        if ((st = upload(p, lut, &p->lut)) != ACCERL_OK) return fail(st);
        p->ingest_arith = fit_ingest_line(lut.data(), &p->ingest_mul, &p->ingest_add) ? 1 : 0;
        p->ingest_shift1 = true;
        for (int u = 0; u < 256; ++u)
            if (lut[u] != (u >> 1)) p->ingest_shift1 = false;
        // the float form of the line (measured faster in the NHWC kernel, slower in the space-to-depth one)
        p->ingest_float = p->ingest_arith == 1 &&
                          fit_ingest_float_line(lut.data(), p->ingest_mul, p->ingest_add, &p->ingest_fa,
                                                &p->ingest_fc1);
    }
    if (value_head) {
        void *d = nullptr;
        const size_t bytes = (size_t)max_batch * p->n_out * sizeof(float) + 256;
        cudaError_t e = cudaMalloc(&d, bytes);
        if (e != cudaSuccess) {
            set_error("create: cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
            cudaGetLastError();
            return fail(e == cudaErrorMemoryAllocation ? ACCERL_ERR_OOM : ACCERL_ERR_CUDA);
        }
        p->owned.push_back(d);
        p->z_scratch = (float *)d;
        p->workspace_bytes += bytes;
    }
    {
        std::vector<int> zero(256, 0);  // word 0 is the status; the rest is trace space
        if ((st = upload(p, zero, &p->status_word)) != ACCERL_OK) return fail(st);
    }
    // ---- launch plan
    {
        Step s0;
        s0.kind = Step::INGEST;
        s0.kernel = in_kind == ACCERL_IN_U8_NCHW ? "ingest_u8_kernel" : "ingest_f32_kernel";
        s0.covers = "ingest";
        p->steps.push_back(s0);
        for (int i = 0; i < n_layers; ++i) {
            Step s;
            s.layer = i;
            s.kind = p->layers[i].kind == ACCERL_CONV2D ? Step::CONV_GENERIC
                     : p->layers[i].kind == ACCERL_FC   ? Step::FC_GENERIC
                                                        : Step::POOL_GENERIC;
            s.kernel = p->layers[i].how;
            s.covers = "layer " + std::to_string(i);
            p->steps.push_back(s);
        }
        Step ss;
        ss.kind = Step::SAMPLE;
        ss.kernel = p->n_actions <= 32 ? "sample_warp_kernel" : "sample_wide_kernel";
        ss.covers = "sample";
        p->steps.push_back(ss);
    }
    p->tensor_s2d.assign(n_layers + 1, 1);
    p->tap_missing.assign(n_layers + 1, 0);
    {
        cudaDeviceProp prop;
        cudaError_t pe = cudaGetDeviceProperties(&prop, device);
        if (pe != cudaSuccess) {
            set_error("create: cudaGetDeviceProperties: %s", cudaGetErrorString(pe));
            return fail(ACCERL_ERR_CUDA);
        }
        p->sm_count = prop.multiProcessorCount;
        if (prop.major != 10) {
            set_error("create: this library is built for sm_100a only (device is sm_%d%d)",
                      prop.major, prop.minor);
            return fail(ACCERL_ERR_UNSUPPORTED);
        }
    }
    if (!(flags & ACCERL_FLAG_FORCE_GENERIC)) {
        bool used = false;
        if ((st = build_tc_plan(p, layers, n_layers, &used)) != ACCERL_OK) return fail(st);
        if (!used && (st = build_tc_mixed_plan(p, layers, n_layers, &used)) != ACCERL_OK)
            return fail(st);
        if (!used && !unfuse_for_taps(p) &&
            (st = build_mlp_plan(p, layers, n_layers, &used)) != ACCERL_OK)
            return fail(st);
    }
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        set_error("create: %s", cudaGetErrorString(e));
        return fail(ACCERL_ERR_CUDA);
    }
    *out = p;
    return ACCERL_OK;
}

accerl_status accerl_policy_act(accerl_policy *p, const void *obs_dev, const float *uniforms_dev,
                                int32_t batch, float *logits_dev, int32_t *actions_dev,
                                float *logp_dev, void *cuda_stream)
{
    accerl_status v = check_act_args(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev,
                                     logp_dev);
    if (v != ACCERL_OK) return v;
    DeviceGuard guard(p->device);
    return run_steps(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev, logp_dev, nullptr, nullptr,
                     (cudaStream_t)cuda_stream, nullptr);
}

accerl_status accerl_policy_act_ex(accerl_policy *p, const void *obs_dev, const float *uniforms_dev,
                                   int32_t batch, float *logits_dev, int32_t *actions_dev,
                                   float *logp_dev, float *value_dev, float *entropy_dev,
                                   void *cuda_stream)
{
    accerl_status v = check_act_args(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev,
                                     logp_dev);
    if (v != ACCERL_OK) return v;
    if (value_dev && p->n_out == p->n_actions) {
        set_error("act_ex: value_dev given but the handle was created without ACCERL_FLAG_VALUE_HEAD");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (((uintptr_t)value_dev & 3) || ((uintptr_t)entropy_dev & 3)) {
        set_error("act_ex: misaligned pointer (value and entropy need 4 bytes)");
        return ACCERL_ERR_INVALID_ARG;
    }
    DeviceGuard guard(p->device);
    return run_steps(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev, logp_dev, value_dev,
                     entropy_dev, (cudaStream_t)cuda_stream, nullptr);
}

accerl_status accerl_policy_act_timed(accerl_policy *p, const void *obs_dev,
                                      const float *uniforms_dev, int32_t batch, float *logits_dev,
                                      int32_t *actions_dev, float *logp_dev, void *cuda_stream,
                                      float *launch_ms_host, int32_t launch_ms_len)
{
    if (!p || !launch_ms_host || launch_ms_len < (int32_t)p->steps.size()) {
        set_error("act_timed: launch_ms_host must hold launches_per_act floats");
        return ACCERL_ERR_INVALID_ARG;
    }
    accerl_status v = check_act_args(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev,
                                     logp_dev);
    if (v != ACCERL_OK) return v;
    DeviceGuard guard(p->device);
    while (p->events.size() < p->steps.size() + 1) {
        cudaEvent_t ev;
        ACCERL_CUDA_TRY(cudaEventCreate(&ev));
        p->events.push_back(ev);
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    v = run_steps(p, obs_dev, uniforms_dev, batch, logits_dev, actions_dev, logp_dev, nullptr, nullptr, st,
                  p->events.data());
    if (v != ACCERL_OK) return v;
    ACCERL_CUDA_TRY(cudaStreamSynchronize(st));
    for (size_t i = 0; i < p->steps.size(); ++i)
        ACCERL_CUDA_TRY(cudaEventElapsedTime(&launch_ms_host[i], p->events[i], p->events[i + 1]));
    return ACCERL_OK;
}

accerl_status accerl_policy_act_host(accerl_policy *p, const void *obs_host,
                                     const float *uniforms_host, int32_t batch,
                                     float *logits_host, int32_t *actions_host, float *logp_host,
                                     void *cuda_stream)
{
    if (!p || !obs_host || !uniforms_host || !logits_host || !actions_host || !logp_host) {
        set_error("act_host: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch < 1) {
        set_error("act_host: batch must be at least 1");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch > p->max_batch) {
        set_error("act_host: batch %d exceeds max_batch %d", batch, p->max_batch);
        return ACCERL_ERR_BATCH_TOO_LARGE;
    }
    DeviceGuard guard(p->device);
    const size_t obs_per_state = (size_t)p->in_c * p->in_h * p->in_w *
                                 (p->in_kind == ACCERL_IN_U8_NCHW ? 1 : sizeof(float));
    if (!p->st_obs) {
        const size_t mb = (size_t)p->max_batch;
        void *d[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
        size_t sz[5] = {obs_per_state * mb, 4 * mb, 4 * mb * (size_t)p->n_actions, 4 * mb, 4 * mb};
        for (int i = 0; i < 5; ++i) {
            ACCERL_CUDA_TRY(cudaMalloc(&d[i], sz[i] + 256));
            p->owned.push_back(d[i]);
            p->workspace_bytes += sz[i] + 256;
        }
        p->st_u = (float *)d[1];
        p->st_logits = (float *)d[2];
        p->st_actions = (int32_t *)d[3];
        p->st_logp = (float *)d[4];
        p->st_obs = d[0];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t B = (size_t)batch;
    // Large batches go in chunks: the host->device copy of chunk i + 1 runs on a stream of its own
    // while chunk i computes (the copy is PCIe-bound and by far the longer part; the chunks only
    // hide the compute and the copies back behind it).  States are independent, so the results are
    // those of one call on the whole batch.
    const int n_chunks = batch >= 4096 ? 8 : 1;
    if (n_chunks > 1 && !p->copy_stream) {
        ACCERL_CUDA_TRY(cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 9; ++i) {
            cudaEvent_t ev;
            ACCERL_CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
            p->copy_events.push_back(ev);
        }
    }
    if (n_chunks == 1) {
        ACCERL_CUDA_TRY(cudaMemcpyAsync(p->st_obs, obs_host, obs_per_state * B, cudaMemcpyHostToDevice, st));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(p->st_u, uniforms_host, 4 * B, cudaMemcpyHostToDevice, st));
        accerl_status s = accerl_policy_act(p, p->st_obs, p->st_u, batch, p->st_logits, p->st_actions,
                                            p->st_logp, cuda_stream);
        if (s != ACCERL_OK) return s;
        ACCERL_CUDA_TRY(cudaMemcpyAsync(logits_host, p->st_logits, 4 * B * p->n_actions,
                                        cudaMemcpyDeviceToHost, st));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(actions_host, p->st_actions, 4 * B, cudaMemcpyDeviceToHost, st));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(logp_host, p->st_logp, 4 * B, cudaMemcpyDeviceToHost, st));
        ACCERL_CUDA_TRY(cudaStreamSynchronize(st));
        return ACCERL_OK;
    }
    // the staging buffers may still be read by earlier work of the caller's stream
    ACCERL_CUDA_TRY(cudaEventRecord(p->copy_events[8], st));
    ACCERL_CUDA_TRY(cudaStreamWaitEvent(p->copy_stream, p->copy_events[8], 0));
    const size_t per = ((B + n_chunks - 1) / n_chunks + 15) & ~(size_t)15;  // keeps every chunk 16-byte aligned
    const size_t A = (size_t)p->n_actions;
    int used = 0;
    for (size_t b0 = 0; b0 < B; b0 += per, ++used) {
        const size_t nb = std::min(per, B - b0);
        ACCERL_CUDA_TRY(cudaMemcpyAsync((char *)p->st_obs + b0 * obs_per_state, (const char *)obs_host + b0 * obs_per_state,
                                        obs_per_state * nb, cudaMemcpyHostToDevice, p->copy_stream));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(p->st_u + b0, uniforms_host + b0, 4 * nb, cudaMemcpyHostToDevice, p->copy_stream));
        ACCERL_CUDA_TRY(cudaEventRecord(p->copy_events[used], p->copy_stream));
    }
    used = 0;
    for (size_t b0 = 0; b0 < B; b0 += per, ++used) {
        const size_t nb = std::min(per, B - b0);
        ACCERL_CUDA_TRY(cudaStreamWaitEvent(st, p->copy_events[used], 0));
        accerl_status s = accerl_policy_act(p, (const char *)p->st_obs + b0 * obs_per_state, p->st_u + b0, (int32_t)nb,
                                            p->st_logits + b0 * A, p->st_actions + b0, p->st_logp + b0, cuda_stream);
        if (s != ACCERL_OK) {
            cudaStreamSynchronize(p->copy_stream);
            return s;
        }
        ACCERL_CUDA_TRY(cudaMemcpyAsync(logits_host + b0 * A, p->st_logits + b0 * A, 4 * nb * A, cudaMemcpyDeviceToHost, st));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(actions_host + b0, p->st_actions + b0, 4 * nb, cudaMemcpyDeviceToHost, st));
        ACCERL_CUDA_TRY(cudaMemcpyAsync(logp_host + b0, p->st_logp + b0, 4 * nb, cudaMemcpyDeviceToHost, st));
    }
    ACCERL_CUDA_TRY(cudaStreamSynchronize(st));
    return ACCERL_OK;
}

accerl_status accerl_policy_read_activation(accerl_policy *p, int32_t layer, int32_t batch,
                                            int8_t *dst, size_t dst_bytes)
{
    if (!p || !dst) {
        set_error("read_activation: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (!(p->flags & ACCERL_FLAG_KEEP_ACTIVATIONS)) {
        set_error("read_activation: the handle was created without ACCERL_FLAG_KEEP_ACTIVATIONS");
        return ACCERL_ERR_INVALID_ARG;
    }
    const int n = (int)p->layers.size();
    if (layer < -1 || layer >= n - 1 || batch < 1 || batch > p->max_batch) {
        set_error("read_activation: layer %d / batch %d out of range", layer, batch);
        return ACCERL_ERR_INVALID_ARG;
    }
    int C, H, W, Cp, buf;
    const int s2 = p->tensor_s2d[layer + 1];
    if (layer < 0) {
        C = p->in_c; H = p->in_h; W = p->in_w; Cp = p->in_cp; buf = p->layers[0].in_buf;
    } else {
        const LayerPlan &L = p->layers[layer];
        C = L.out_c; H = L.out_h; W = L.out_w; Cp = L.out_cp; buf = L.out_buf;
    }
    const size_t need = (size_t)batch * C * H * W;
    if (dst_bytes < need) {
        set_error("read_activation: destination holds %zu bytes, %zu needed", dst_bytes, need);
        return ACCERL_ERR_INVALID_ARG;
    }
    if (p->tap_missing[layer + 1]) {
        set_error("read_activation: the fused plan never stores tensor %d", layer);
        return ACCERL_ERR_UNSUPPORTED;
    }
    DeviceGuard guard(p->device);
    if ((size_t)(layer + 1) < p->taps.size() && p->taps[layer + 1].ptr) {
        // the tensor is only stored with a zero border and a fixed pixel pitch
        const TapDesc &t = p->taps[layer + 1];
        std::vector<int8_t> pad;
        try {
            pad.resize((size_t)batch * t.hpitch * t.wpitch * t.pitch);
        } catch (...) {
            set_error("read_activation: out of host memory");
            return ACCERL_ERR_OOM;
        }
        ACCERL_CUDA_TRY(cudaDeviceSynchronize());
        ACCERL_CUDA_TRY(cudaMemcpy(pad.data(), t.ptr, pad.size(), cudaMemcpyDeviceToHost));
        for (int b = 0; b < batch; ++b)
            for (int c = 0; c < C; ++c)
                for (int y = 0; y < H; ++y)
                    for (int x = 0; x < W; ++x)
                        dst[(((size_t)b * C + c) * H + y) * W + x] =
                            pad[(((size_t)b * t.hpitch + y + t.off_y) * t.wpitch + x + t.off_x) * t.pitch + c];
        return ACCERL_OK;
    }
    std::vector<int8_t> tmp;
    try {
        tmp.resize((size_t)batch * H * W * Cp);
    } catch (...) {
        set_error("read_activation: out of host memory");
        return ACCERL_ERR_OOM;
    }
    ACCERL_CUDA_TRY(cudaDeviceSynchronize());
    ACCERL_CUDA_TRY(cudaMemcpy(tmp.data(), p->bufs[buf].ptr, tmp.size(), cudaMemcpyDeviceToHost));
    for (int b = 0; b < batch; ++b)
        for (int c = 0; c < C; ++c)
            for (int y = 0; y < H; ++y)
                for (int x = 0; x < W; ++x)
                    dst[(((size_t)b * C + c) * H + y) * W + x] =
                        tmp[((((size_t)b * (H / s2) + y / s2) * (W / s2) + x / s2) * s2 * s2 +
                             (y % s2) * s2 + x % s2) * Cp + c];
    return ACCERL_OK;
}

accerl_status accerl_policy_check(accerl_policy *p)
{
    if (!p) {
        set_error("check: null handle");
        return ACCERL_ERR_INVALID_ARG;
    }
    DeviceGuard guard(p->device);
    ACCERL_CUDA_TRY(cudaStreamSynchronize(p->last_stream));
    int word = 0;
    ACCERL_CUDA_TRY(cudaMemcpy(&word, p->status_word, sizeof(int), cudaMemcpyDeviceToHost));
    if (word != 0) {
        set_error("check: a device-side bounded wait gave up (status word 0x%x)", word);
        int zero = 0;
        cudaMemcpy(p->status_word, &zero, sizeof(int), cudaMemcpyHostToDevice);
        return ACCERL_ERR_TIMEOUT;
    }
    return ACCERL_OK;
}

accerl_status accerl_policy_info(const accerl_policy *p, int32_t batch, int32_t *n_actions,
                                 size_t *workspace_bytes, int32_t *launches_per_act,
                                 char *plan_buf, size_t plan_buf_bytes)
{
    if (!p) {
        set_error("info: null handle");
        return ACCERL_ERR_INVALID_ARG;
    }
    (void)batch;
    if (n_actions) *n_actions = p->n_actions;
    if (workspace_bytes) *workspace_bytes = p->workspace_bytes;
    std::string s;
    char line[320];
    int launches = 0;
    for (const Step &t : p->steps) {
        if (t.layer >= 0) {
            const LayerPlan &L = p->layers[t.layer];
            snprintf(line, sizeof(line), "launch %d: %s covers %s (%s %dx%dx%d -> %dx%dx%d)\n",
                     launches, t.kernel.c_str(), t.covers.c_str(),
                     L.kind == ACCERL_CONV2D ? "conv" : (L.kind == ACCERL_FC ? "fc" : "maxpool"),
                     L.in_c, L.in_h, L.in_w, L.out_c, L.out_h, L.out_w);
        } else {
            snprintf(line, sizeof(line), "launch %d: %s covers %s\n", launches, t.kernel.c_str(),
                     t.covers.c_str());
        }
        s += line;
        ++launches;
    }
    if (!p->plan_note.empty()) s += "note: " + p->plan_note + "\n";
    if (launches_per_act) *launches_per_act = launches;
    if (plan_buf && plan_buf_bytes) {
        size_t n = std::min(plan_buf_bytes - 1, s.size());
        memcpy(plan_buf, s.data(), n);
        plan_buf[n] = 0;
    }
    return ACCERL_OK;
}

#ifdef ACCERL_TC_TRACE
// traced builds only: copy out and clear the per-launch role stopwatches (8 counters per launch)
accerl_status accerl_debug_read_trace(accerl_policy *p, unsigned long long *out, int n)
{
    cudaDeviceSynchronize();
    cudaMemcpy(out, p->status_word + 16, n * 8, cudaMemcpyDeviceToHost);
    cudaMemset(p->status_word + 16, 0, n * 8);
    return ACCERL_OK;
}
#endif

}  // extern "C"
