// Tensor-core plan for residual conv stacks (the IMPALA-ResNet shape): 3x3 stride-1 pad-1
// convolutions with 16 or 32 channels run on tc_gemm_kernel in shifted mode, a first conv on
// 4-channel frames too, max-pools on a CUDA-core kernel.
//
// Wide images (W >= 16), "slot" layout: a tensor is stored [n][H+2][PW][C] with the image at row 1,
// pixel 1, zero elsewhere, PW a multiple of 8 >= W + 2.  One GEMM row is P consecutive stored
// pixels (P * C_in = 64 or 128 bytes) and produces the P output pixels above them, N = P * C_out
// = 128 columns, with banded weights: output pixel j of the row meets stored pixels j .. j + 2 of
// the rows of the three taps ky, i.e. the P pixels of the GEMM row ky * PW/P further down plus the
// first two of the row after it.  The K loop is the list of the 32-byte steps that cover those
// (P + 2) * C_in bytes; most of the weight matrix is zero, but with 16 or 32 output channels the
// tensor pipe is paid per instruction, not per flop, and a tile of 128 x 128 outputs amortises
// the epilogue's per-tile work eight times better than 128 x 16.
//
// Narrow images, "pad" layout: [n][H+2][W+2][32 bytes] (channels 16..31 zero when the tensor has
// 16), one GEMM row per padded position, taps at row offsets ky * (W+2) + kx, one K step per tap.
//
// Borders and padding are zeroed once at create and never written.  A tensor may be kept in two
// forms at once (for instance the input x of a residual block: as it is for the skip add, and
// ReLU'd for the block's first conv); producers (the conv epilogue, the pooling kernel) write both.
#include <string.h>

#include <algorithm>

#include "epilogue.cuh"
#include "internal.h"

namespace accerl {

// ---------------------------------------------------------------------------------------
// max-pool with up to two stored forms of its output (any pitches and offsets, optionally ReLU'd)
// ---------------------------------------------------------------------------------------
__global__ void maxpool_dual_kernel(const PoolDualParams q, long long total)
{
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int G = q.C / 16;  // 16-byte channel groups per pixel
    int g, ox, oy;
    long long n;
    if (total < (1LL << 31)) {  // 32-bit divisions: a quarter of the instructions of the 64-bit ones
        unsigned t = (unsigned)idx;
        g = (int)(t % (unsigned)G);
        t /= (unsigned)G;
        ox = (int)(t % (unsigned)q.OW);
        t /= (unsigned)q.OW;
        oy = (int)(t % (unsigned)q.OH);
        n = t / (unsigned)q.OH;
    } else {
        g = (int)(idx % G);
        long long t = idx / G;
        ox = (int)(t % q.OW);
        t /= q.OW;
        oy = (int)(t % q.OH);
        n = t / q.OH;
    }
    uint32_t m[4] = {0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u};
    const int8_t *win = q.in + ((n * q.in_hpitch + oy * q.stride + q.in_off_y) * q.in_wpitch + ox * q.stride_x +
                                q.in_off_x) * q.C + g * 16;
    const int row_bytes = q.in_wpitch * q.C;
    auto take = [&](int ky, int kx) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(win + ky * row_bytes + kx * q.C));
        m[0] = __vmaxs4(m[0], v.x);
        m[1] = __vmaxs4(m[1], v.y);
        m[2] = __vmaxs4(m[2], v.z);
        m[3] = __vmaxs4(m[3], v.w);
    };
    if (q.k == 3 && q.kw == 3) {
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) take(ky, kx);
    } else if (q.k == 3 && q.kw == 1) {  // the producer has already pooled along x
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) take(ky, 0);
    } else {
        for (int ky = 0; ky < q.k; ++ky)
            for (int kx = 0; kx < q.kw; ++kx) take(ky, kx);
    }
#pragma unroll
    for (int o = 0; o < 2; ++o) {
        const PoolOut &po = q.out[o];
        if (!po.ptr) continue;
        uint4 v = make_uint4(m[0], m[1], m[2], m[3]);
        if (po.relu) v = make_uint4(__vmaxs4(m[0], 0u), __vmaxs4(m[1], 0u), __vmaxs4(m[2], 0u), __vmaxs4(m[3], 0u));
        *reinterpret_cast<uint4 *>(po.ptr + ((n * po.hpitch + oy + po.off_y) * po.wpitch + ox + po.off_x) * po.pix_bytes +
                                   g * 16) = v;
    }
}

cudaError_t launch_maxpool_dual(const PoolDualParams &q, int B, cudaStream_t st)
{
    const long long total = (long long)B * q.OH * q.OW * (q.C / 16);
    maxpool_dual_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(q, total);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// uint8 NCHW frames with 4 channels -> plain int8 NHWC: four pixels per thread
// ---------------------------------------------------------------------------------------
template <int ARITH>
__global__ void ingest_u8_nhwc4_kernel(const uint8_t *__restrict__ obs, const int8_t *__restrict__ lut,
                                       int8_t *__restrict__ out, long long total, int H, int W4,
                                       int out_hpitch, int out_wpitch, int off_y, int off_x,
                                       uint32_t mul, uint32_t add)
{
    __shared__ int8_t s_lut[256];
    if (!ARITH) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = lut[i];
        __syncthreads();
    }
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    // idx = (n * H + y) * W4 + x4: pixels 4*x4 .. 4*x4+3 of row y of image n (W is a multiple of 4)
    int x4, y;
    long long n;
    if (total < (1LL << 31)) {  // 32-bit divisions where the count allows
        unsigned t = (unsigned)idx;
        x4 = (int)(t % (unsigned)W4);
        t /= (unsigned)W4;
        y = (int)(t % (unsigned)H);
        n = t / (unsigned)H;
    } else {
        x4 = (int)(idx % W4);
        long long t = idx / W4;
        y = (int)(t % H);
        n = t / H;
    }
    const int W = 4 * W4;
    uint32_t plane[4];
#pragma unroll
    for (int c = 0; c < 4; ++c)
        plane[c] = __ldg(reinterpret_cast<const uint32_t *>(obs + ((n * 4 + c) * H + y) * W) + x4);
    uint32_t w[4];
    if (ARITH == 4) {  // the table is u >> 1: four bytes at a time, then a 4 x 4 byte transpose
        const uint4 v = ingest_shift_line16(plane[0], plane[1], plane[2], plane[3]);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    } else
#pragma unroll
    for (int px = 0; px < 4; ++px) {
        if (ARITH == 2) {
            w[px] = ingest_float_line4(plane[0], plane[1], plane[2], plane[3], px, __uint_as_float(mul),
                                       __uint_as_float(add));
        } else if (ARITH == 1) {
            uint32_t pr[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) pr[c] = ((plane[c] >> (8 * px)) & 0xff) * mul + add;
            const uint32_t lo = __byte_perm(pr[0], pr[1], 0x0073), hi = __byte_perm(pr[2], pr[3], 0x0073);
            w[px] = __vminu4(__byte_perm(lo, hi, 0x5410), 0x7f7f7f7fu);
        } else {
            uint32_t word = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                word |= (uint32_t)(uint8_t)s_lut[(plane[c] >> (8 * px)) & 0xff] << (8 * c);
            w[px] = word;
        }
    }
    // off_x is a multiple of 4 pixels, so the 16-byte store stays aligned
    *reinterpret_cast<uint4 *>(out + (((n * out_hpitch + y + off_y) * out_wpitch) + 4 * x4 + off_x) * 4LL) =
        make_uint4(w[0], w[1], w[2], w[3]);
}

cudaError_t launch_ingest_u8_nhwc4(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int H, int W,
                                   int out_hpitch, int out_wpitch, int off_y, int off_x, int arith,
                                   uint32_t mul, uint32_t add, cudaStream_t st)
{
    const long long total = (long long)B * H * (W / 4);
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (arith == 4)
        ingest_u8_nhwc4_kernel<4><<<blocks, 256, 0, st>>>(obs, lut, out, total, H, W / 4, out_hpitch,
                                                         out_wpitch, off_y, off_x, mul, add);
    else if (arith == 2)
        ingest_u8_nhwc4_kernel<2><<<blocks, 256, 0, st>>>(obs, lut, out, total, H, W / 4, out_hpitch,
                                                         out_wpitch, off_y, off_x, mul, add);
    else if (arith == 1)
        ingest_u8_nhwc4_kernel<1><<<blocks, 256, 0, st>>>(obs, lut, out, total, H, W / 4, out_hpitch,
                                                         out_wpitch, off_y, off_x, mul, add);
    else
        ingest_u8_nhwc4_kernel<0><<<blocks, 256, 0, st>>>(obs, lut, out, total, H, W / 4, out_hpitch,
                                                         out_wpitch, off_y, off_x, mul, add);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// plan
// ---------------------------------------------------------------------------------------
namespace {

enum Role { GENERIC, POOL, TCCONV, TCPX, TCFC, TCFIRST };

struct Forms {  // which stored forms of a tensor its readers need
    bool plain = false, plain_relu = false, pad = false, pad_relu = false, slot = false, slot_relu = false;
    bool hp = false;  // pooled along x by its producer: [n][H][hp_w][C], read by a max-pool only
    int8_t *p_plain = nullptr, *p_plain_relu = nullptr, *p_pad = nullptr, *p_slot = nullptr,
           *p_slot_relu = nullptr, *p_hp = nullptr;
    int count() const
    {
        return (plain ? 1 : 0) + (plain_relu ? 1 : 0) + ((pad || pad_relu) ? 1 : 0) + (slot ? 1 : 0) +
               (slot_relu ? 1 : 0) + (hp ? 1 : 0);
    }
};

int slot_pw(int W) { return round_up(W + 2, 8); }

// pixels per GEMM row of a multi-pixel conv, 0 if the layer does not qualify
int tcpx_pixels(const accerl_layer_desc &d)
{
    if (d.kind != ACCERL_CONV2D || d.kh != 3 || d.kw != 3 || d.stride != 1 || d.pad != 1) return 0;
    if ((d.in_c != 16 && d.in_c != 32) || (d.out_c != 16 && d.out_c != 32) || d.in_w < 16) return 0;
    const int P = 128 / d.out_c, row = P * d.in_c;
    if (row != 64 && row != 128) return 0;
    if (128 + 2 * (slot_pw(d.in_w) / P) + 1 > 248) return 0;
    return P;
}

bool tcconv_ok(const accerl_layer_desc &d)
{
    return d.kind == ACCERL_CONV2D && d.kh == 3 && d.kw == 3 && d.stride == 1 && d.pad == 1 &&
           (d.in_c == 16 || d.in_c == 32) && d.out_c % 16 == 0 && d.out_c <= 256 &&
           128 + 2 * (d.in_w + 2) + 2 <= 256;
}

// stored pixels per row of a tensor that its producer (P pixels per GEMM row) has pooled along x
int hp_width(int W, int P) { return slot_pw(W) / P * (P / 2); }

accerl_status alloc_zeroed(accerl_policy *p, size_t bytes, int8_t **out)
{
    void *d = nullptr;
    ACCERL_CUDA_TRY(cudaMalloc(&d, bytes + 4096));  // slack: TMA boxes may start before the tail
    p->owned.push_back(d);
    p->workspace_bytes += bytes + 4096;
    ACCERL_CUDA_TRY(cudaMemset(d, 0, bytes + 4096));
    *out = (int8_t *)d;
    return ACCERL_OK;
}

}  // namespace

accerl_status build_tc_mixed_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                                  bool *used)
{
    *used = false;
    if (p->in_kind != ACCERL_IN_U8_NCHW) return ACCERL_OK;
    const bool keep = unfuse_for_taps(p);  // every tensor must exist in an un-ReLU'd form
    const bool tap_fused = (p->flags & ACCERL_FLAG_TAP_FUSED) != 0;
    // ---- roles
    std::vector<Role> role(n_layers);
    int n_tc = 0;
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        const LayerPlan &L = p->layers[i];
        if (tcconv_ok(d)) {
            role[i] = tcpx_pixels(d) ? TCPX : TCCONV;
            ++n_tc;
        } else if (d.kind == ACCERL_MAXPOOL && (d.in_c == 16 || d.in_c == 32) && d.pad == 0) {
            role[i] = POOL;
        } else if (d.kind == ACCERL_FC) {
            const int K = L.in_h * L.in_w * L.in_cp;
            const bool fits = L.in_cp == L.in_c && K % 16 == 0 && K >= 128 &&
                              (K + 127) / 128 <= kTcMaxChunks &&
                              ((d.flags & ACCERL_LOGITS) ? d.out_c <= 256
                                                         : (d.out_c % 16 == 0 && d.out_c <= kTcMaxN &&
                                                            (d.out_c <= 256 || d.out_c % 256 == 0)));
            if (!fits && !fc_sample_fits(p, layers, n_layers, i)) return ACCERL_OK;
            role[i] = TCFC;
        } else if (d.kind == ACCERL_CONV2D && d.skip_from < 0 && i == 0) {
            // A first conv on 4-channel frames: tensor cores if its only reader is a max-pool (see
            // the TCFIRST branch below), else the dp4a kernel.
            const bool toeplitz = d.in_c == 4 && d.kh == 3 && d.kw == 3 && d.stride == 1 && d.pad == 1 &&
                                  (d.out_c == 16 || d.out_c == 32) && d.in_w % 4 == 0 && n_layers > 1 &&
                                  layers[1].kind == ACCERL_MAXPOOL && !(d.flags & ACCERL_RELU_IN);
            role[i] = toeplitz ? TCFIRST : GENERIC;
        } else {
            return ACCERL_OK;
        }
        if (d.skip_from >= 0 && role[i] != TCCONV && role[i] != TCPX) return ACCERL_OK;
    }
    if (n_tc == 0) return ACCERL_OK;
    for (int i = 0; i < n_layers; ++i)
        if ((long long)p->max_batch * (p->layers[i].in_h + 2) * (p->layers[i].in_w + 2) + 512 >= (1LL << 31))
            return ACCERL_OK;

    // A multi-pixel conv cannot write the pad layout of a 16-channel tensor (its pixels are not
    // contiguous there): such a layer falls back to one position per GEMM row.
    for (int i = 0; i + 1 < n_layers; ++i)
        if (role[i] == TCPX && role[i + 1] == TCCONV) role[i] = TCCONV;

    // ---- forms of every tensor (index t + 1; tensor -1 is the quantised input)
    std::vector<Forms> forms(n_layers + 1);
    forms[0].plain = true;  // the input feeds the generic first conv
    if (role[0] != GENERIC && role[0] != TCFIRST) return ACCERL_OK;
    for (int j = 1; j < n_layers; ++j)
        if (layers[j].skip_from == 0 && role[0] == TCFIRST) role[0] = GENERIC;  // tensor 0 must be pool-only
    for (int j = 1; j < n_layers; ++j) {
        const accerl_layer_desc &d = layers[j];
        Forms &f = forms[j];  // tensor j - 1
        const bool relu_in = (d.flags & ACCERL_RELU_IN) && !(layers[j - 1].flags & ACCERL_RELU_OUT);
        if (role[j] == GENERIC) {
            if (relu_in) return ACCERL_OK;
            f.plain = true;
        } else if (role[j] == POOL) {
            if (relu_in) return ACCERL_OK;
            // a pool reads whatever its producer writes naturally
            // a pool reads whatever its producer writes naturally; a multi-pixel conv that only feeds
            // a 3x3 stride-2 pool pools along x itself (TcGemmParams::hpool)
            bool only_reader = !keep && j >= 1 && role[j - 1] == TCPX && d.kh == 3 && d.kw == 3 &&
                               d.stride == 2 && d.pad == 0 && layers[j - 1].skip_from < 0;
            for (int q = 0; q < n_layers && only_reader; ++q)
                if (layers[q].skip_from == j - 1) only_reader = false;
            if (only_reader) {
                const int P = tcpx_pixels(layers[j - 1]);
                // (measured: worth it while the wider K window still fits four 32-byte steps per tap row)
                only_reader = (P / 2) * (layers[j - 1].out_c / 16) == 4 && (P + 1) * layers[j - 1].out_c <= 256 &&
                              (P + 3) * layers[j - 1].in_c <= 128;
            }
            if (only_reader) f.hp = true;
            else (role[j - 1] == TCPX ? f.slot : f.plain) = true;
        } else if (role[j] == TCCONV) {
            (relu_in ? f.pad_relu : f.pad) = true;
        } else if (role[j] == TCPX) {
            (relu_in ? f.slot_relu : f.slot) = true;
        } else {
            (relu_in ? f.plain_relu : f.plain) = true;
        }
        if (d.skip_from >= 0) {
            Forms &fs = forms[d.skip_from + 1];
            (role[j] == TCPX ? fs.slot : fs.plain) = true;
        }
    }
    for (int t = 0; t < n_layers; ++t) {
        Forms &f = forms[t];
        if (f.pad && f.pad_relu) return ACCERL_OK;
        if (keep && !f.plain && !f.pad && !f.slot) f.plain = true;  // the parity tap needs an un-ReLU'd form
        if (f.count() > 2) return ACCERL_OK;
        if (t > 0 && (role[t - 1] == GENERIC || role[t - 1] == TCFIRST) && (f.count() != 1 || !f.plain))
            return ACCERL_OK;
        if (t > 0 && role[t - 1] == TCPX && (f.pad || f.pad_relu) && layers[t - 1].out_c != 32)
            return ACCERL_OK;
    }

    // ---- buffers: plain forms live in the generic plan's buffers, the others are new
    accerl_status st;
    for (int t = 0; t < n_layers; ++t) {
        Forms &f = forms[t];
        const int C = t == 0 ? p->in_cp : p->layers[t - 1].out_cp;
        const int H = t == 0 ? p->in_h : p->layers[t - 1].out_h;
        const int W = t == 0 ? p->in_w : p->layers[t - 1].out_w;
        if (f.plain) f.p_plain = t == 0 ? p->bufs[p->layers[0].in_buf].ptr
                                        : p->bufs[p->layers[t - 1].out_buf].ptr;
        if (f.plain_relu &&
            (st = alloc_zeroed(p, (size_t)p->max_batch * H * W * C, &f.p_plain_relu)) != ACCERL_OK)
            return st;
        if ((f.pad || f.pad_relu) &&
            (st = alloc_zeroed(p, (size_t)p->max_batch * (H + 2) * (W + 2) * 32, &f.p_pad)) != ACCERL_OK)
            return st;
        const size_t slot_bytes = (size_t)p->max_batch * (H + 2) * slot_pw(W) * C;
        if (f.hp && (st = alloc_zeroed(p, (size_t)p->max_batch * H * hp_width(W, tcpx_pixels(layers[t - 1])) * C,
                                       &f.p_hp)) != ACCERL_OK)
            return st;
        if (f.slot && (st = alloc_zeroed(p, slot_bytes, &f.p_slot)) != ACCERL_OK) return st;
        if (f.slot_relu && (st = alloc_zeroed(p, slot_bytes, &f.p_slot_relu)) != ACCERL_OK) return st;
    }

    // ---- first conv on tensor cores: frames stored as [n][H+2][PW][4 B] with the image at row 1,
    // pixel 4, PW a multiple of 8 pixels, so that 8 pixels form one 32-byte GEMM row; its output is
    // plain NHWC with rows of OW8 * 8 pixels
    const int W0 = p->in_w, H0 = p->in_h;
    const int PW = round_up(4 + W0 + 1, 8), PW8 = PW / 8, OW8 = (W0 + 7) / 8;
    // Without the parity taps the first conv pools along x on its accumulators (TcGemmParams::hpool)
    // and stores [n][H][OW8 * 4][C]: 4 pooled pixels per GEMM row.
    const bool hpool_first = role[0] == TCFIRST && !keep && layers[0].out_c == 16 && layers[1].kh == 3 &&
                             layers[1].kw == 3 && layers[1].stride == 2 && layers[1].pad == 0;
    const int first_wpitch = hpool_first ? OW8 * 4 : OW8 * 8;
    int8_t *first_out = nullptr;
    if (role[0] == TCFIRST) {
        if ((st = alloc_zeroed(p, (size_t)p->max_batch * (H0 + 2) * PW * 4, &p->in_pad4)) != ACCERL_OK)
            return st;
        p->in_pad4_w = PW;
        if ((st = alloc_zeroed(p, (size_t)p->max_batch * H0 * first_wpitch * layers[0].out_c, &first_out)) !=
            ACCERL_OK)
            return st;
    }

    // ---- steps
    auto bail = [&]() {  // the generic plan stays: forget everything built so far
        p->taps.clear();
        p->pools.clear();
        p->tc_steps.clear();
        return ACCERL_OK;
    };
    std::vector<Step> steps;
    bool fused_sample = false;
    p->taps.assign(n_layers + 1, TapDesc());
    {
        Step s0;
        const bool fast = p->in_c == 4 && p->in_w % 4 == 0;
        s0.kind = role[0] == TCFIRST ? Step::INGEST_PAD4 : (fast ? Step::INGEST_NHWC4 : Step::INGEST);
        s0.kernel = fast ? "ingest_u8_nhwc4_kernel" : "ingest_u8_kernel";
        if (role[0] == TCFIRST) {
            TapDesc &td = p->taps[0];
            td.ptr = p->in_pad4;
            td.pitch = 4;
            td.hpitch = H0 + 2;
            td.wpitch = PW;
            td.off_y = 1;
            td.off_x = 4;
        }
        s0.covers = "ingest";
        steps.push_back(s0);
    }
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        const LayerPlan &L = p->layers[i];
        const Forms &fin = forms[i], &fout = forms[i + 1];
        Step s;
        s.layer = i;
        s.covers = "layer " + std::to_string(i);
        if (i + 1 < n_layers && !fout.plain && fout.pad) {
            // parity tap from the padded, un-ReLU'd form
            TapDesc &td = p->taps[i + 1];
            td.ptr = fout.p_pad;
            td.pitch = 32;
            td.hpitch = L.out_h + 2;
            td.wpitch = L.out_w + 2;
            td.off_y = td.off_x = 1;
        } else if (i + 1 < n_layers && !fout.plain && fout.slot) {
            TapDesc &td = p->taps[i + 1];
            td.ptr = fout.p_slot;
            td.pitch = L.out_cp;
            td.hpitch = L.out_h + 2;
            td.wpitch = slot_pw(L.out_w);
            td.off_y = td.off_x = 1;
        }
        if (role[i] == GENERIC) {
            s.kind = Step::CONV_GENERIC;
            s.kernel = L.how;
            steps.push_back(s);
            continue;
        }
        if (role[i] == POOL) {
            PoolDualParams q;
            memset(&q, 0, sizeof(q));
            if (i == 1 && role[0] == TCFIRST) {
                q.in = first_out;
                q.in_hpitch = L.in_h;
                q.in_wpitch = first_wpitch;
            } else if (fin.hp) {
                q.in = fin.p_hp;
                q.in_hpitch = L.in_h;
                q.in_wpitch = hp_width(L.in_w, tcpx_pixels(layers[i - 1]));
            } else if (fin.slot) {
                q.in = fin.p_slot;
                q.in_hpitch = L.in_h + 2;
                q.in_wpitch = slot_pw(L.in_w);
                q.in_off_y = q.in_off_x = 1;
            } else {
                q.in = fin.p_plain;
                q.in_hpitch = L.in_h;
                q.in_wpitch = L.in_w;
            }
            int n_po = 0;
            const int OH = L.out_h, OW = L.out_w, C = L.in_c;
            if (fout.plain) q.out[n_po++] = PoolOut{fout.p_plain, OH, OW, 0, 0, C, 0};
            if (fout.plain_relu) q.out[n_po++] = PoolOut{fout.p_plain_relu, OH, OW, 0, 0, C, 1};
            if ((fout.pad || fout.pad_relu) && n_po < 2)
                q.out[n_po++] = PoolOut{fout.p_pad, OH + 2, OW + 2, 1, 1, 32, fout.pad_relu ? 1 : 0};
            else if (fout.pad || fout.pad_relu) return bail();
            if (fout.slot && n_po < 2) q.out[n_po++] = PoolOut{fout.p_slot, OH + 2, slot_pw(OW), 1, 1, C, 0};
            else if (fout.slot) return bail();
            if (fout.slot_relu && n_po < 2)
                q.out[n_po++] = PoolOut{fout.p_slot_relu, OH + 2, slot_pw(OW), 1, 1, C, 1};
            else if (fout.slot_relu) return bail();
            q.H = L.in_h; q.W = L.in_w; q.C = L.in_c; q.OH = L.out_h; q.OW = L.out_w;
            q.k = d.kh; q.stride = d.stride;
            const bool pre_pooled = (hpool_first && i == 1) || fin.hp;
            q.kw = pre_pooled ? 1 : d.kw;
            q.stride_x = pre_pooled ? 1 : d.stride;
            p->pools.push_back(q);
            s.kind = Step::POOL_DUAL;
            s.tc = (int)p->pools.size() - 1;
            s.kernel = "maxpool_dual_kernel";
            steps.push_back(s);
            continue;
        }
        if (role[i] == TCFC && fin.plain && fc_sample_fits(p, layers, n_layers, i)) {
            // the last layer runs fused with the sampler
            if ((st = build_fc_sample(p, d, i, fin.p_plain, L.in_c, &s)) != ACCERL_OK) return st;
            steps.push_back(s);
            fused_sample = true;
            continue;
        }
        // ---- tensor-core layer
        TcStep ts;
        memset(&ts.prm, 0, sizeof(ts.prm));
        TcGemmParams &g = ts.prm;
        const bool logits = (d.flags & ACCERL_LOGITS) != 0;
        const int P = role[i] == TCPX ? tcpx_pixels(d) : 0;  // stored pixels per GEMM row
        const bool hp_out = role[i] == TCPX && fout.hp;       // pools along x: one output pixel more per row
        const int Pout = hp_out ? P + 1 : P;
        const int first_px = hpool_first ? 9 : 8;  // output pixels per GEMM row of the first conv
        const int n_total = role[i] == TCFIRST ? first_px * d.out_c : (P ? Pout * d.out_c : round_up(d.out_c, 16));
        g.sub = 1;
        g.max_sub = 1;
        g.out_xmul = g.out2_xmul = 1;
        g.n_total = n_total;
        g.n_tile = n_total > 256 ? 256 : n_total;
        if (d.kind == ACCERL_FC && !logits) {
            // small batches: narrower tiles, so that the weight stream is shared by more SMs
            const int m_tiles = (p->max_batch + 127) / 128;
            while (g.n_tile > 32 && g.n_tile % 32 == 0 && 2 * m_tiles * (n_total / g.n_tile) <= p->sm_count)
                g.n_tile /= 2;
        }
        g.n_tiles = n_total / g.n_tile;
        std::vector<int8_t> packed;
        const int8_t *a_ptr;
        long long a_rows_total;
        int row_bytes;
        const float *ks_dev = L.kscale, *bs_dev = L.bias;
        const int32_t *px_skip_mul = nullptr;
        if (role[i] == TCFIRST) {
            // GEMM row = 8 consecutive padded pixels (32 B); output column j * out_c + oc is output
            // pixel j of the group.  Input pixel (row ky, offset d8 * 8 + pin from the group's
            // first pixel) meets tap kx = d8 * 8 + pin - j - 3 of output pixel j.
            g.chunk_bytes = 32;
            g.n_chunks = 6;
            g.rows_per_image = (H0 + 2) * PW8;
            g.grid_w = PW8;
            g.shifted = 1;
            g.a_rows = round_up(128 + 2 * PW8 + 1, 8);
            packed.assign((size_t)6 * n_total * 32, 0);
            for (int ky = 0; ky < 3; ++ky)
                for (int d8 = 0; d8 < 2; ++d8) {
                    const int j = ky * 2 + d8;
                    g.row_off[j] = ky * PW8 + d8;
                    g.col_off[j] = 0;
                    for (int px = 0; px < first_px; ++px)
                        for (int oc = 0; oc < d.out_c; ++oc)
                            for (int pin = 0; pin < 8; ++pin) {
                                const int kx = d8 * 8 + pin - px - 3;
                                if (kx < 0 || kx > 2) continue;
                                for (int c = 0; c < 4; ++c)
                                    packed[((size_t)j * n_total + px * d.out_c + oc) * 32 + pin * 4 + c] =
                                        d.w[((oc * 4 + c) * 3 + ky) * 3 + kx];
                            }
                }
            a_ptr = p->in_pad4;
            a_rows_total = (long long)p->max_batch * (H0 + 2) * PW8;
            row_bytes = 32;
            // per-column scales: the channel's, repeated for the pixels of the row
            std::vector<float> ks(n_total), bs(n_total);
            for (int px = 0; px < first_px; ++px)
                for (int oc = 0; oc < d.out_c; ++oc) {
                    volatile float k = d.s_in * d.s_w[oc];
                    ks[px * d.out_c + oc] = k;
                    bs[px * d.out_c + oc] = d.bias[oc];
                }
            void *kd = nullptr, *bd = nullptr;
            if ((st = upload_bytes(p, ks.data(), ks.size() * 4, &kd)) != ACCERL_OK) return st;
            if ((st = upload_bytes(p, bs.data(), bs.size() * 4, &bd)) != ACCERL_OK) return st;
            ks_dev = (const float *)kd;
            bs_dev = (const float *)bd;
        } else if (role[i] == TCPX) {
            // GEMM row = P stored pixels; its K window is those and the next two pixels, for each
            // of the three rows ky: steps of 32 bytes, the last one or two from the GEMM row after.
            const int PW = slot_pw(d.in_w), G = PW / P, row = P * d.in_c;
            const int first_ks = row / 32, n_ks = ((Pout + 2) * d.in_c + 31) / 32;
            g.chunk_bytes = row;
            g.kstep_list = 1;
            g.n_chunks = 3 * n_ks;
            g.rows_per_image = (d.in_h + 2) * G;
            g.grid_w = G;
            g.shifted = 1;
            g.a_rows = round_up(128 + 2 * G + 2, 8);
            g.px_per_row = P;
            g.px_cols = d.out_c;
            g.px_w = d.in_w;
            packed.assign((size_t)g.n_chunks * n_total * 32, 0);
            for (int ky = 0; ky < 3; ++ky)
                for (int ks = 0; ks < n_ks; ++ks) {
                    const int j = ky * n_ks + ks;
                    g.row_off[j] = ky * G + (ks < first_ks ? 0 : 1);
                    g.col_off[j] = 32 * (ks < first_ks ? ks : ks - first_ks);
                    for (int px = 0; px < Pout; ++px)
                        for (int oc = 0; oc < d.out_c; ++oc)
                            for (int kk = 0; kk < 32; ++kk) {
                                const int wb = 32 * ks + kk, pin = wb / d.in_c, c = wb % d.in_c;
                                const int kx = pin - px;
                                if (kx < 0 || kx > 2) continue;
                                packed[((size_t)j * n_total + px * d.out_c + oc) * 32 + kk] =
                                    d.w[((oc * d.in_c + c) * 3 + ky) * 3 + kx];
                            }
                }
            const bool relu_in = (d.flags & ACCERL_RELU_IN) && !(layers[i - 1].flags & ACCERL_RELU_OUT);
            a_ptr = relu_in ? fin.p_slot_relu : fin.p_slot;
            a_rows_total = (long long)p->max_batch * (d.in_h + 2) * G;
            row_bytes = row;
            // per-column scales and residual multipliers: the channel's, repeated for the P pixels
            std::vector<float> ks(n_total), bs(n_total);
            std::vector<int32_t> sm(n_total, 0);
            for (int px = 0; px < Pout; ++px)
                for (int oc = 0; oc < d.out_c; ++oc) {
                    volatile float k = d.s_in * d.s_w[oc];
                    ks[px * d.out_c + oc] = k;
                    bs[px * d.out_c + oc] = d.bias[oc];
                    if (d.skip_from >= 0) sm[px * d.out_c + oc] = d.skip_mul[oc];
                }
            void *kd = nullptr, *bd = nullptr, *sd = nullptr;
            if ((st = upload_bytes(p, ks.data(), ks.size() * 4, &kd)) != ACCERL_OK) return st;
            if ((st = upload_bytes(p, bs.data(), bs.size() * 4, &bd)) != ACCERL_OK) return st;
            if ((st = upload_bytes(p, sm.data(), sm.size() * 4, &sd)) != ACCERL_OK) return st;
            ks_dev = (const float *)kd;
            bs_dev = (const float *)bd;
            px_skip_mul = (const int32_t *)sd;
        } else if (role[i] == TCCONV) {
            const int Hp = d.in_h + 2, Wp = d.in_w + 2;
            g.chunk_bytes = 32;
            g.n_chunks = 9;
            g.rows_per_image = Hp * Wp;
            g.grid_w = Wp;
            g.shifted = 1;
            g.max_sub = 2;
            g.a_rows = round_up(128 + 2 * Wp + 2, 8);
            packed.assign((size_t)9 * n_total * 32, 0);
            for (int ky = 0; ky < 3; ++ky)
                for (int kx = 0; kx < 3; ++kx) {
                    const int j = ky * 3 + kx;
                    g.row_off[j] = ky * Wp + kx;
                    g.col_off[j] = 0;
                    for (int oc = 0; oc < d.out_c; ++oc)
                        for (int c = 0; c < d.in_c; ++c)
                            packed[((size_t)j * n_total + oc) * 32 + c] =
                                d.w[((oc * d.in_c + c) * 3 + ky) * 3 + kx];
                }
            a_ptr = fin.p_pad;
            a_rows_total = (long long)p->max_batch * Hp * Wp;
            row_bytes = 32;
        } else {
            const int K = L.in_h * L.in_w * L.in_cp;
            g.chunk_bytes = 128;
            g.n_chunks = (K + 127) / 128;
            g.rows_per_image = 1;
            g.grid_w = 1;
            packed.assign((size_t)g.n_chunks * n_total * 128, 0);
            for (int j = 0; j < g.n_chunks; ++j) {
                g.row_off[j] = 0;
                g.col_off[j] = 128 * j;
            }
            for (int oc = 0; oc < d.out_c; ++oc)
                for (int c = 0; c < L.in_c; ++c)
                    for (int y = 0; y < L.in_h; ++y)
                        for (int x = 0; x < L.in_w; ++x) {
                            const int ki = (y * L.in_w + x) * L.in_cp + c;
                            packed[((size_t)(ki / 128) * n_total + oc) * 128 + ki % 128] =
                                d.w[(size_t)oc * d.in_c + (c * L.in_h + y) * L.in_w + x];
                        }
            const bool relu_in = (d.flags & ACCERL_RELU_IN) && !(layers[i - 1].flags & ACCERL_RELU_OUT);
            a_ptr = relu_in ? fin.p_plain_relu : fin.p_plain;
            a_rows_total = p->max_batch;
            row_bytes = K;
        }
        g.out_h = L.out_h;
        g.out_w = role[i] == TCFIRST ? OW8 : L.out_w;
        g.out_s2d = 1;
        g.out_s2d_log2 = 0;
        g.inv_rows_per_image = 1.0f / (float)g.rows_per_image;
        g.grid_w_magic = g.grid_w == 1 ? 0xffffffffu : (unsigned)(((1ULL << 32) + g.grid_w - 1) / g.grid_w);
        // outputs: every stored form of tensor i
        struct OutSpec {
            int8_t *ptr;
            int rpi, gw, off, pitch, relu, xmul;
        } outs[4];
        int n_out = 0;
        if (role[i] == TCFIRST) {
            if (hpool_first) {  // in pooled pixels; no tap (the un-pooled tensor is never stored)
                outs[n_out++] = OutSpec{first_out, L.out_h * first_wpitch, first_wpitch, 0, d.out_c, 0, 4};
            } else {
                outs[n_out++] = OutSpec{first_out, L.out_h * OW8, OW8, 0, n_total, 0, 1};
                TapDesc &td = p->taps[i + 1];
                td.ptr = first_out;
                td.pitch = d.out_c;
                td.hpitch = L.out_h;
                td.wpitch = OW8 * 8;
            }
        } else if (!logits) {
            // Row pitch = one pixel of the stored form; a multi-pixel GEMM row starts at pixel
            // X * P and its columns run on over the following pixels.
            const int H = L.out_h, W = L.out_w, xm = P ? P : 1, px = P ? d.out_c : n_total;
            const int SW = slot_pw(W);
            if (fout.plain) outs[n_out++] = OutSpec{fout.p_plain, H * W, W, 0, px, 0, xm};
            if (fout.plain_relu) outs[n_out++] = OutSpec{fout.p_plain_relu, H * W, W, 0, px, 1, xm};
            if (fout.pad || fout.pad_relu) {
                if (P && d.out_c != 32) return bail();
                outs[n_out++] = OutSpec{fout.p_pad, (H + 2) * (W + 2), W + 2, W + 3, 32, fout.pad_relu ? 1 : 0, xm};
            }
            if (fout.hp) {
                const int hw = hp_width(W, P);
                outs[n_out++] = OutSpec{fout.p_hp, H * hw, hw, 0, L.out_cp, 0, P / 2};
            }
            if (fout.slot) outs[n_out++] = OutSpec{fout.p_slot, (H + 2) * SW, SW, SW + 1, L.out_cp, 0, xm};
            if (fout.slot_relu)
                outs[n_out++] = OutSpec{fout.p_slot_relu, (H + 2) * SW, SW, SW + 1, L.out_cp, 1, xm};
        }
        if (!logits) {
            if (n_out == 0 || n_out > 2) return bail();
            g.out = outs[0].ptr;
            g.out_rows_per_image = outs[0].rpi;
            g.out_grid_w = outs[0].gw;
            g.out_row_off = outs[0].off;
            g.out_pitch = outs[0].pitch;
            g.out_relu = outs[0].relu;
            g.out_xmul = outs[0].xmul;
            if (n_out == 2) {
                g.out2 = outs[1].ptr;
                g.out2_rows_per_image = outs[1].rpi;
                g.out2_grid_w = outs[1].gw;
                g.out2_row_off = outs[1].off;
                g.out2_pitch = outs[1].pitch;
                g.out2_relu = outs[1].relu;
                g.out2_xmul = outs[1].xmul;
            }
        }
        if (d.skip_from >= 0) {
            const Forms &fs = forms[d.skip_from + 1];
            g.skip_pitch = p->layers[d.skip_from].out_cp;
            if (P) {
                const int SW = slot_pw(L.out_w);
                g.skip = fs.p_slot;
                g.skip_mul = px_skip_mul;
                g.skip_rows_per_image = (L.out_h + 2) * SW;
                g.skip_grid_w = SW;
                g.skip_xmul = P;
                g.skip_row_off = SW + 1;
            } else {
                g.skip = fs.p_plain;
                g.skip_mul = L.skip_mul;
                g.skip_rows_per_image = L.out_h * L.out_w;
                g.skip_grid_w = L.out_w;
                g.skip_xmul = 1;
                g.skip_row_off = 0;
            }
            if (!g.skip) return bail();
        }
        g.kscale = ks_dev;
        g.bias = bs_dev;
        g.s_out = L.s_out;
        g.relu_out = (d.flags & ACCERL_RELU_OUT) != 0;
        {
            volatile float inv = 1.0f / L.s_out;
            g.inv_s_out = inv;
        }
        // the single-fma requantiser where every channel has verified constants (searched first: a layer
        // that has them needs no check of the three-step division)
        if (!logits && !(p->flags & ACCERL_FLAG_TEST_NO_FASTDIV) && !(p->flags & ACCERL_FLAG_TEST_NO_AFFINE)) {
            const bool repeated = role[i] == TCFIRST || P;  // columns = (pixel of the row, channel)
            std::vector<float> kh(n_total, 0.f), bh(n_total, 0.f), k2, b2;
            for (int j = 0; j < n_total; ++j) {
                const int oc = repeated ? j % d.out_c : j;
                if (oc >= d.out_c) continue;
                volatile float k = d.s_in * d.s_w[oc];
                kh[j] = k;
                bh[j] = d.bias[oc];
            }
            bool ok = false;
            st = fit_affine_requant(kh.data(), bh.data(), n_total, g.s_out, g.relu_out != 0, &k2, &b2, &ok);
            if (st != ACCERL_OK) return st;
            if (ok) {
                void *kd = nullptr, *bd = nullptr;
                if ((st = upload_bytes(p, k2.data(), k2.size() * 4, &kd)) != ACCERL_OK) return st;
                if ((st = upload_bytes(p, b2.data(), b2.size() * 4, &bd)) != ACCERL_OK) return st;
                g.kscale = (const float *)kd;
                g.bias = (const float *)bd;
                g.affine = 1;
                g.fast_div = 1;  // a verified division-free requantiser exists
            }
        }
        if (!logits && !g.affine) {
            float kmax = 0.f, bmax = 0.f;
            for (int c = 0; c < d.out_c; ++c) {
                kmax = std::max(kmax, d.s_in * d.s_w[c]);
                bmax = std::max(bmax, fabsf(d.bias[c]));
            }
            st = choose_fastdiv(g.s_out, g.relu_out != 0, 2147483648.0f * kmax + bmax,
                                !(p->flags & ACCERL_FLAG_TEST_NO_FASTDIV), &g.inv_s_out, &g.fast_div);
            if (st != ACCERL_OK) return st;
        }
        g.split_cols = (g.n_tile > 128 || (role[i] == TCFIRST && hpool_first) || hp_out) ? 1 : 0;
        // (a multi-pixel layer whose output scale fails the division check keeps its place in the plan:
        // its launch runs the epilogue that re-does elements near a rounding tie with the IEEE divide)
        if (hp_out) {
            g.hpool = 1;
            g.px_w = (L.out_w - 3) / 2 + 1;  // pooled width
        }
        if (role[i] == TCFIRST && hpool_first) {
            g.hpool = 1;
            g.px_per_row = 8;  // selects the multi-pixel kernel
            g.px_cols = d.out_c;
            g.px_w = (W0 - 3) / 2 + 1;  // pooled width
        }
        // Multi-pixel layers with 128-byte output rows collect the 32 rows of a warp in shared memory and
        // move whole 128-byte lines: a lane's 16-byte pieces would each touch a line of their own, and
        // the load/store path then bounds the layer (residual layers 872 -> 574 us, plain 16 -> 16
        // layers at 41 x 41 330-360 -> 260 us)
        g.staged = (role[i] == TCPX && g.n_tile == 128) ? 1 : 0;
        g.logits_mode = logits ? 1 : 0;
        g.n_actions = p->n_out;  // columns of the fp32 rows the logits layer writes
        g.status = p->status_word;
        g.trace_slot = (int)p->tc_steps.size() % 8;
        const int b_bytes = g.kstep_list ? 32 : g.chunk_bytes;  // bytes of a weight row per chunk
        ts.resident_b = g.n_tiles == 1 && (size_t)g.n_chunks * n_total * b_bytes <= 112 * 1024;
        if (g.shifted && !ts.resident_b) return bail();
        if (!tc_choose_pipeline(g, ts.resident_b)) {
            if (g.shifted) return bail();
            ts.resident_b = false;
            if (!tc_choose_pipeline(g, false)) return bail();
        }
        void *w_dev = nullptr;
        if ((st = upload_bytes(p, packed.data(), packed.size(), &w_dev)) != ACCERL_OK) return st;
        if ((st = tc_make_map(ts.map_a, a_ptr, a_rows_total, row_bytes, row_bytes,
                              g.shifted ? g.a_rows : 128, g.chunk_bytes)) != ACCERL_OK)
            return st;
        if ((st = tc_make_map(ts.map_b, w_dev, (long long)g.n_chunks * n_total, b_bytes, b_bytes, g.n_tile,
                              b_bytes)) != ACCERL_OK)
            return st;
        p->tc_steps.push_back(ts);
        s.kind = Step::TC_GEMM;
        s.tc = (int)p->tc_steps.size() - 1;
        s.kernel = ts.resident_b ? "tc_gemm_kernel<resident weights>" : "tc_gemm_kernel<streamed weights>";
        if (g.fast_div) s.kernel += g.affine ? "[single-fma requantiser verified]" : "[3-step divide verified]";
        else if (!logits) s.kernel += "[division check failed: exact divide near ties]";
        if (g.hpool) s.kernel += "[pooled along x on the accumulators]";
        steps.push_back(s);
    }
    if (!fused_sample) {
        Step ss;
        ss.kind = Step::SAMPLE;
        ss.kernel = p->n_actions <= 32 ? "sample_warp_kernel" : "sample_wide_kernel";
        ss.covers = "sample";
        steps.push_back(ss);
    }
    if (tap_fused) {
        // tensors the fused plan stores in no un-ReLU'd form cannot be tapped
        for (int t = 1; t <= n_layers - 1; ++t) {
            const Forms &f = forms[t];
            p->tap_missing[t] = !(f.plain || f.pad || f.slot) ? 1 : 0;
        }
        if (hpool_first) p->tap_missing[1] = 1;
    }
    p->steps = steps;
    *used = true;
    return ACCERL_OK;
}

}  // namespace accerl
