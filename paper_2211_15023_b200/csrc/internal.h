// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <memory>
#include <string>
#include <vector>

#include "accerl.h"
#include "tc_conv.h"
#include "tc_conv1.h"
#include "tc_gemm.h"

namespace accerl {

void set_error(const char *fmt, ...);

#define ACCERL_CUDA_TRY(expr)                                                              \
    do {                                                                                   \
        cudaError_t e_ = (expr);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            ::accerl::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e_),    \
                                __FILE__, __LINE__);                                       \
            return e_ == cudaErrorMemoryAllocation ? ACCERL_ERR_OOM : ACCERL_ERR_CUDA;     \
        }                                                                                  \
    } while (0)

static inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// One layer as the kernels see it.  Activations live in device memory as NHWC int8 with the
// channel count padded to a multiple of 4 (`*_cp`), so that four channels form one 32-bit word.
struct LayerPlan {
    int kind = 0;
    uint32_t flags = 0;
    int in_c = 0, in_h = 0, in_w = 0, out_c = 0, out_h = 0, out_w = 0;
    int kh = 0, kw = 0, stride = 1, pad = 0;
    int in_cp = 0, out_cp = 0;
    float s_in = 1.f, s_out = 1.f;
    int skip_from = -1;
    int in_buf = -1, out_buf = -1, skip_buf = -1;  // indices into accerl_policy::bufs
    // device parameters
    int32_t *w_generic = nullptr;  // conv: [tap][in_cp/4][oc_pad] words; fc: [oc_pad][K/4]
    float *kscale = nullptr;       // [oc_pad]  s_in * s_w[c], 0 for padding channels
    float *bias = nullptr;         // [oc_pad]
    int32_t *skip_mul = nullptr;   // [oc_pad] or null
    int oc_pad = 0;                // out_c rounded up to 16
    std::string how;               // which kernel serves the layer (for accerl_policy_info)
};

// One kernel launch of the plan: which kernel, and which part of the path it covers
// ("ingest", "layer 3", "layers 3-4", "sample", joined by '+').
struct Step {
    enum Kind { INGEST, CONV_GENERIC, FC_GENERIC, POOL_GENERIC, SAMPLE, INGEST_S2D, TC_GEMM, MLP_FUSED,
                INGEST_NHWC4, POOL_DUAL, INGEST_PAD4, FC_SAMPLE, CONV1_FRAMES, CONV_ROWS } kind;
    int layer = -1;
    int tc = -1;  // index into accerl_policy::tc_steps (TC_GEMM), ::pools (POOL_DUAL) or ::conv_rows (CONV_ROWS)
    std::string kernel, covers;
};

// One launch of the tensor-core contraction: TMA descriptors (built once, for max_batch rows) and
// the parameter block; batch-dependent fields are filled in per call.
struct TcStep {
    alignas(64) unsigned char map_a[128];
    alignas(64) unsigned char map_b[128];
    TcGemmParams prm;
    bool resident_b = false;
};

// One launch of the strided-conv kernel (tc_conv.cu)
struct ConvRowsStep {
    alignas(64) unsigned char map_a[128];
    alignas(64) unsigned char map_b[128];
    ConvRowsParams prm;
};

struct MlpFusedParams;  // mlp_fused.cu

// last FC layer fused with the sampler (fc_sample.cu)
struct FcSampleParams {
    const int8_t *x;  // [B][pitch] int8 input rows
    int pitch, k4, n_actions;
    int n_out;         // output columns: n_actions, or n_actions + 1 with a value head
    const int32_t *w;  // [k4][32] words, lane = output column
    const float *kscale, *bias;
};

// max-pool that writes a plain NHWC output and / or a padded-border one (tc_mixed_plan.cu)
struct PoolOut {  // one stored form of the pooled tensor
    int8_t *ptr;                 // null: unused
    int hpitch, wpitch;          // stored rows per image, pixels per stored row
    int off_y, off_x;            // where pixel (0, 0) sits
    int pix_bytes;               // bytes between stored pixels (>= C)
    int relu;                    // store max(code, 0)
};
struct PoolDualParams {
    const int8_t *in;            // pixels of C bytes
    int in_hpitch, in_wpitch, in_off_y, in_off_x;
    int H, W, C, OH, OW, k, stride;
    int kw, stride_x;  // window width and horizontal stride (k and stride when the input is not pre-pooled)
    PoolOut out[2];
};

// where the parity tap of a tensor lives when it is not in the generic plan's buffer
struct TapDesc {
    const int8_t *ptr = nullptr;
    int pitch = 0;               // bytes per stored pixel
    int hpitch = 0, wpitch = 0;  // stored rows per image, pixels per stored row
    int off_y = 0, off_x = 0;    // where pixel (0, 0) sits
};

struct DeviceBuf {
    int8_t *ptr = nullptr;
    size_t bytes_per_state = 0;
};

}  // namespace accerl

struct accerl_policy {
    int device = 0;
    int in_kind = 0;
    int in_c = 0, in_h = 0, in_w = 0, in_cp = 0;
    float s_input = 1.f;
    int max_batch = 0;
    uint32_t flags = 0;
    int n_actions = 0;
    int n_out = 0;                        // columns of the last layer: n_actions (+ 1 with a value head)
    float *z_scratch = nullptr;           // device [max_batch][n_out]: last layer's floats when the
                                          // plan's sampler is a launch of its own and n_out != n_actions
    std::vector<accerl::LayerPlan> layers;
    std::vector<accerl::Step> steps;      // the launch sequence of one act call
    std::string plan_note;                // why a faster plan was not taken (shown by accerl_policy_info)
    std::vector<accerl::TcStep> tc_steps;
    std::vector<accerl::PoolDualParams> pools;
    std::vector<accerl::ConvRowsStep> conv_rows;
    accerl::Conv1Params conv1 = {};       // used by a Step::CONV1_FRAMES launch
    alignas(64) unsigned char conv1_map_b[128] = {};
    int8_t *in_pad4 = nullptr;            // frames as [n][H+2][PW][4] with the image at (1, 4)
    int in_pad4_w = 0;
    std::vector<accerl::TapDesc> taps;    // per tensor (index t + 1); empty or null ptr = generic buffer
    std::vector<char> tap_missing;        // per tensor (index t + 1): the plan never stores it (TAP_FUSED)
    std::shared_ptr<accerl::MlpFusedParams> mlp;  // set when the whole step is one fused launch
    accerl::FcSampleParams fc_sample = {};         // used by a Step::FC_SAMPLE launch
    std::vector<int> tensor_s2d;          // space-to-depth factor of tensor t at [t + 1]
    int sm_count = 0;
    std::vector<accerl::DeviceBuf> bufs;  // bufs[0] holds the quantised input
    int8_t *lut = nullptr;                // device, 256-entry uint8 -> int8 input table
    int ingest_arith = 0;                 // the table is the line min((u * mul + add) >> 24, 127)
    uint32_t ingest_mul = 0, ingest_add = 0;
    bool ingest_shift1 = false;           // the table is exactly u >> 1 (s_input = 1/127)
    bool ingest_float = false;            // the same line in float form: code = low byte of fma(f - c1, A, 1.5 * 2^23)
    uint32_t ingest_fa = 0, ingest_fc1 = 0;  // bit patterns of A and c1
    int *status_word = nullptr;           // device, set by kernels whose bounded waits give up
    size_t workspace_bytes = 0;
    std::vector<void *> owned;            // every device allocation, for destroy
    cudaStream_t last_stream = nullptr;
    std::vector<cudaEvent_t> events;      // steps.size() + 1 events, created on first timed call
    // host-call staging (allocated on first accerl_policy_act_host)
    void *st_obs = nullptr;
    float *st_u = nullptr, *st_logits = nullptr, *st_logp = nullptr;
    int32_t *st_actions = nullptr;
    cudaStream_t copy_stream = nullptr;   // host->device copies of chunked accerl_policy_act_host calls
    std::vector<cudaEvent_t> copy_events; // one per chunk, and one for the caller's stream
    // the quantised parameters accerl_policy_create_fp32 computed (empty for other handles)
    struct PtqLayer {
        std::vector<int8_t> w;
        std::vector<float> s_w;
        std::vector<int32_t> skip_mul;
        float s_in = 1.f, s_out = 1.f;
    };
    std::vector<PtqLayer> ptq;
    // outputs of this policy inside accerl_policy_act_mixed (allocated on its first call)
    float *mix_logits = nullptr, *mix_logp = nullptr, *mix_value = nullptr, *mix_entropy = nullptr;
    int32_t *mix_actions = nullptr;
};

namespace accerl {

// KEEP_ACTIVATIONS without TAP_FUSED: build the plan whose every tensor exists
static inline bool unfuse_for_taps(const accerl_policy *p)
{
    return (p->flags & ACCERL_FLAG_KEEP_ACTIVATIONS) && !(p->flags & ACCERL_FLAG_TAP_FUSED);
}

// generic CUDA-core kernels (generic_kernels.cu); every launcher enqueues on `st` and returns
// the launch status
cudaError_t launch_ingest_u8(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int C,
                             int H, int W, int Cp, cudaStream_t st);
cudaError_t launch_ingest_f32(const float *obs, float s_input, int8_t *out, int B, int D, int Dp,
                              cudaStream_t st);
cudaError_t launch_conv_generic(const LayerPlan &L, const int8_t *in, const int8_t *skip,
                                int8_t *out, int B, cudaStream_t st);
cudaError_t launch_fc_generic(const LayerPlan &L, const int8_t *in, int8_t *out, float *logits,
                              int B, cudaStream_t st);
cudaError_t launch_maxpool_generic(const LayerPlan &L, const int8_t *in, int8_t *out, int B,
                                   cudaStream_t st);
cudaError_t launch_sample(const float *z, int pitch, const float *u, int B, int A, float *logits_out,
                          int32_t *actions, float *logp, float *value, float *entropy, cudaStream_t st);

// tensor-core plan (tc_plan.cu): replaces p->steps when the whole network qualifies; returns
// ACCERL_OK with *used = false when it does not
accerl_status build_tc_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                            bool *used);
// mixed tensor-core / CUDA-core plan for residual 3x3 conv stacks (tc_mixed_plan.cu)
accerl_status build_tc_mixed_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                                  bool *used);
cudaError_t launch_maxpool_dual(const PoolDualParams &q, int B, cudaStream_t st);
cudaError_t launch_ingest_u8_nhwc4(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int H, int W,
                                   int out_hpitch, int out_wpitch, int off_y, int off_x, int arith,
                                   uint32_t mul, uint32_t add, cudaStream_t st);
// single-launch plan for all-FC policies on vector observations (mlp_fused.cu)
accerl_status build_mlp_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                             bool *used);
cudaError_t launch_mlp_fused(const accerl_policy *p, const float *obs, const float *u, int B,
                             float *logits, int32_t *actions, float *logp, float *value, float *entropy,
                             cudaStream_t st);
accerl_status upload_bytes(accerl_policy *p, const void *host, size_t bytes, void **dev);
bool fc_sample_fits(const accerl_policy *p, const accerl_layer_desc *layers, int n_layers, int i);
accerl_status build_fc_sample(accerl_policy *p, const accerl_layer_desc &d, int layer, const int8_t *x,
                              int pitch, Step *out);
cudaError_t launch_fc_sample(const FcSampleParams &q, const float *u, int B, float *logits,
                             int32_t *actions, float *logp, float *value, float *entropy, int sm_count,
                             cudaStream_t st);

}  // namespace accerl
