// accerl_policy_act_noalloc: the Actor step for callers that must not allocate device memory.
//
// The activation workspace of this variant is a fixed array inside the library image instead of
// buffers obtained from cudaMalloc.  See the declaration in accerl.h for who needs it and why.
#include <mutex>

#include "internal.h"

namespace {

constexpr size_t kScratchBytes = ACCERL_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Reserved on every GPU on which this library's CUDA module gets loaded, until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char *g_scratch_dev[kMaxDevices];  // device address of the array, per device; null = not yet asked

struct CurrentDevice {
    int prev = -1;
    bool ok;
    explicit CurrentDevice(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~CurrentDevice()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can
// use: ask the runtime once per device (with that device current) where the array lives there.
accerl_status scratch_on(int device, unsigned char **out)
{
    if (device < 0 || device >= kMaxDevices) {
        accerl::set_error("act_noalloc: device index %d not supported (0..%d)", device,
                          kMaxDevices - 1);
        return ACCERL_ERR_UNSUPPORTED;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_dev[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) {
            accerl::set_error("act_noalloc: cudaGetSymbolAddress failed on device %d: %s", device,
                              cudaGetErrorString(e));
            cudaGetLastError();
            return ACCERL_ERR_CUDA;
        }
        g_scratch_dev[device] = (unsigned char *)ptr;
    }
    *out = g_scratch_dev[device];
    return ACCERL_OK;
}

}  // namespace

using namespace accerl;

extern "C" accerl_status accerl_policy_act_noalloc(accerl_policy *p, const void *obs_dev,
                                                   const float *uniforms_dev, int32_t batch,
                                                   float *logits_dev, int32_t *actions_dev,
                                                   float *logp_dev, void *cuda_stream)
{
    if (!p || !obs_dev || !uniforms_dev || !logits_dev || !actions_dev || !logp_dev) {
        set_error("act_noalloc: null argument");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (batch < 1) {
        set_error("act_noalloc: batch must be at least 1");
        return ACCERL_ERR_INVALID_ARG;
    }
    if (((uintptr_t)obs_dev & 15) || ((uintptr_t)uniforms_dev & 3) || ((uintptr_t)logits_dev & 3) ||
        ((uintptr_t)actions_dev & 3) || ((uintptr_t)logp_dev & 3)) {
        set_error("act_noalloc: misaligned pointer (obs needs 16 bytes, the others 4)");
        return ACCERL_ERR_INVALID_ARG;
    }
    // carve the handle's logical buffers out of the fixed array
    constexpr int kMaxBufs = 64;
    size_t offset[kMaxBufs];
    if (p->bufs.size() > (size_t)kMaxBufs) {
        set_error("act_noalloc: the policy needs %zu workspace buffers (at most %d supported)",
                  p->bufs.size(), kMaxBufs);
        return ACCERL_ERR_UNSUPPORTED;
    }
    size_t total = 0;
    for (size_t b = 0; b < p->bufs.size(); ++b) {
        offset[b] = total;
        size_t bytes = p->bufs[b].bytes_per_state * (size_t)batch;
        total += (bytes + 255) / 256 * 256;
    }
    // a value head: the last layer's rows (logits, then V) pass through the array as well
    const size_t z_offset = total;
    if (p->n_out != p->n_actions) total += ((size_t)batch * p->n_out * sizeof(float) + 255) / 256 * 256;
    if (total > kScratchBytes) {
        set_error("act_noalloc: batch %d needs %zu bytes of activation workspace, the built-in "
                  "scratch holds %zu (use accerl_policy_act, or a smaller batch)",
                  batch, total, kScratchBytes);
        return ACCERL_ERR_BATCH_TOO_LARGE;
    }
    CurrentDevice cur(p->device);
    if (!cur.ok) {
        set_error("act_noalloc: cudaSetDevice(%d) failed", p->device);
        return ACCERL_ERR_CUDA;
    }
    unsigned char *base = nullptr;
    accerl_status s = scratch_on(p->device, &base);
    if (s != ACCERL_OK) return s;
    auto buf = [&](int b) { return (int8_t *)(base + offset[b]); };

    cudaStream_t st = (cudaStream_t)cuda_stream;
    p->last_stream = st;  // accerl_policy_check waits for this step
    const int B = batch;
    float *z_dev = p->n_out != p->n_actions ? (float *)(base + z_offset) : logits_dev;
    int8_t *x = buf(p->layers[0].in_buf);
    if (p->in_kind == ACCERL_IN_U8_NCHW)
        ACCERL_CUDA_TRY(launch_ingest_u8((const uint8_t *)obs_dev, p->lut, x, B, p->in_c, p->in_h,
                                         p->in_w, p->in_cp, st));
    else
        ACCERL_CUDA_TRY(launch_ingest_f32((const float *)obs_dev, p->s_input, x, B, p->in_c,
                                          p->in_cp, st));
    for (const LayerPlan &L : p->layers) {
        const int8_t *in = buf(L.in_buf);
        int8_t *o = L.out_buf >= 0 ? buf(L.out_buf) : nullptr;
        if (L.kind == ACCERL_CONV2D)
            ACCERL_CUDA_TRY(launch_conv_generic(L, in, L.skip_buf >= 0 ? buf(L.skip_buf) : nullptr, o,
                                                B, st));
        else if (L.kind == ACCERL_FC)
            ACCERL_CUDA_TRY(launch_fc_generic(L, in, o, z_dev, B, st));
        else
            ACCERL_CUDA_TRY(launch_maxpool_generic(L, in, o, B, st));
    }
    ACCERL_CUDA_TRY(launch_sample(z_dev, p->n_out, uniforms_dev, B, p->n_actions,
                                  z_dev != logits_dev ? logits_dev : nullptr, actions_dev, logp_dev,
                                  nullptr, nullptr, st));
    return ACCERL_OK;
}
