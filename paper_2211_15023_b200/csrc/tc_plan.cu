// Builds the tensor-core plan of a policy: which activation layouts the layers exchange, how the
// weights are packed for the shifted-row implicit GEMM, the TMA descriptors and launch
// parameters.  Also holds the input kernel that writes frames in space-to-depth form.
#include <string.h>

#include <algorithm>
#include <mutex>

#include "epilogue.cuh"
#include "internal.h"

namespace accerl {

// ---------------------------------------------------------------------------------------
// uint8 NCHW frames -> int8 space-to-depth(s) rows, C = 4, s = 4: each thread turns one 4 x 4
// pixel block of all four channel planes into one 64-byte output row ((dy, dx, c) order).
// With ARITH the table lookup is replaced by q = min((u * mul + add) >> 24, 127), a fixed-point
// line that the host has checked against all 256 table entries; the product fits 32 bits, so the
// code is simply the top byte of the multiply-add.
// ---------------------------------------------------------------------------------------
template <int ARITH>
__global__ void ingest_u8_s2d44_kernel(const uint8_t *__restrict__ obs,
                                       const int8_t *__restrict__ lut, uint4 *__restrict__ out,
                                       int B, int H, int W, uint32_t mul, uint32_t add)
{
    __shared__ int8_t s_lut[256];
    if (!ARITH) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s_lut[i] = lut[i];
        __syncthreads();
    }
    // One block = one image, one thread = one output row (Y, X); all index arithmetic is 32-bit
    // and per image (the kernel is bound by integer instructions, not by memory).  Sixteen
    // independent 4-byte loads (4 image rows of 4 channel planes) are in flight before the first
    // is used, then 64 contiguous bytes are stored.
    const int Ws = W / 4, rows = (H / 4) * Ws;
    const int pos = blockIdx.y * blockDim.x + threadIdx.x;
    if (pos >= rows) return;
    const int n = blockIdx.x;
    const int Y = pos / Ws, X = pos - Y * Ws;
    const uint8_t *img = obs + (size_t)n * 4 * H * W + (4 * Y) * W + 4 * X;
    const long long idx = (long long)n * rows + pos;
    const int plane_bytes = H * W;
    uint32_t plane[4][4];  // [dy][c]
#pragma unroll
    for (int dy = 0; dy < 4; ++dy)
#pragma unroll
        for (int c = 0; c < 4; ++c)
            plane[dy][c] = __ldg(reinterpret_cast<const uint32_t *>(img + c * plane_bytes + dy * W));
#pragma unroll
    for (int dy = 0; dy < 4; ++dy) {
        uint32_t w[4];
#pragma unroll
        for (int dx = 0; dx < 4; ++dx) {
            if (ARITH == 2) {
                w[dx] = ingest_float_line4(plane[dy][0], plane[dy][1], plane[dy][2], plane[dy][3], dx,
                                           __uint_as_float(mul), __uint_as_float(add));
            } else if (ARITH == 1) {
                uint32_t pr[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) pr[c] = ((plane[dy][c] >> (8 * dx)) & 0xff) * mul + add;
                // top bytes of the four products, channel 0 in the low byte
                const uint32_t lo = __byte_perm(pr[0], pr[1], 0x0073);
                const uint32_t hi = __byte_perm(pr[2], pr[3], 0x0073);
                w[dx] = __vminu4(__byte_perm(lo, hi, 0x5410), 0x7f7f7f7fu);
            } else {
                uint32_t word = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    word |= (uint32_t)(uint8_t)s_lut[(plane[dy][c] >> (8 * dx)) & 0xff] << (8 * c);
                w[dx] = word;
            }
        }
        out[idx * 4 + dy] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// any C, s: one thread per output byte
__global__ void ingest_u8_s2d_any_kernel(const uint8_t *__restrict__ obs,
                                         const int8_t *__restrict__ lut, int8_t *__restrict__ out,
                                         long long total, int C, int H, int W, int s)
{
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int Ws = W / s, Hs = H / s, Cs = s * s * C;
    int b = (int)(idx % Cs);
    long long r = idx / Cs;
    int X = (int)(r % Ws);
    r /= Ws;
    int Y = (int)(r % Hs);
    long long n = r / Hs;
    int c = b % C, dx = (b / C) % s, dy = b / (C * s);
    out[idx] = lut[obs[((n * C + c) * H + s * Y + dy) * W + s * X + dx]];
}

// Fit q(u) = min((u * mul + add) >> 24, 127) to a 256-entry input table; false if no line fits.
bool fit_ingest_line(const int8_t *lut, uint32_t *mul, uint32_t *add)
{
    int last = 255;  // entries from the first 127 on may be clamped
    for (int u = 0; u < 256; ++u) {
        if (lut[u] < 0) return false;
        if (lut[u] == 127) {
            last = u;
            break;
        }
    }
    if (last < 2) return false;
    const long long one = 1LL << 24;
    const double slope = (double)lut[last] / last;
    const long long a0 = (long long)(slope * one);
    for (long long a = a0 - 4096; a <= a0 + 4096; ++a) {
        if (a <= 0) continue;
        long long lo = 0, hi = one * 256;  // add in [lo, hi)
        for (int u = 0; u < 256 && lo < hi; ++u) {
            const long long q = lut[u];
            lo = std::max(lo, q * one - u * a);
            if (u < last) hi = std::min(hi, (q + 1) * one - u * a);
        }
        hi = std::min(hi, (1LL << 32) - 255 * a);  // the multiply-add must not wrap
        if (lo < hi) {
            const long long b = lo + (hi - lo) / 2;
            bool ok = true;
            for (int u = 0; u < 256 && ok; ++u) {
                const unsigned long long v = (unsigned long long)u * a + b;
                ok = v < (1ULL << 32) && std::min<long long>((long long)(v >> 24), 127) == lut[u];
            }
            if (ok) {
                *mul = (uint32_t)a;
                *add = (uint32_t)b;
                return true;
            }
        }
    }
    return false;
}

// The same table as a float line (see ingest_float_line4 in epilogue.cuh): byte u becomes the float
// 128 + u/256 by a byte permute, g = that - c1, r = fma(g, A, 1.5 * 2^23), and the code is the low
// byte of r's bit pattern.  Starting from the fixed-point line, a few offsets are tried and each
// candidate is run through exactly the device's float operations for all 256 inputs.
bool fit_ingest_float_line(const int8_t *lut, uint32_t mul, uint32_t add, uint32_t *a_bits, uint32_t *c1_bits)
{
    const double one = 16777216.0, m = (double)mul / one;
    for (int i = 0; i < 256; ++i)
        if (lut[i] < 0) return false;
    for (int t = -8; t <= 8; ++t) {
        const double k = (double)add / one - 0.5 + t * 2.5e-4;  // floor(x) = rint(x - 1/2) off the ties
        const float A = (float)(256.0 * m);
        const float c1 = (float)(128.0 - k / (double)A);
        bool ok = true;
        for (int u = 0; u < 256 && ok; ++u) {
            uint32_t fb = 0x43000000u | ((uint32_t)u << 8), rb;
            float f, r;
            memcpy(&f, &fb, 4);
            volatile float g = f - c1;
            r = fmaf(g, A, 12582912.0f);
            memcpy(&rb, &r, 4);
            ok = (rb & 0xffu) == (uint32_t)lut[u] && r >= 12582912.0f && r < 12582912.0f + 128.0f;
        }
        if (ok) {
            memcpy(a_bits, &A, 4);
            memcpy(c1_bits, &c1, 4);
            return true;
        }
    }
    return false;
}

cudaError_t launch_ingest_u8_s2d(const uint8_t *obs, const int8_t *lut, int8_t *out, int B, int C,
                                 int H, int W, int s, int arith, uint32_t mul, uint32_t add,
                                 cudaStream_t st)
{
    if (C == 4 && s == 4 && W % 4 == 0) {
        const int rows = (H / 4) * (W / 4), threads = rows >= 448 ? 224 : 128;
        const dim3 grid((unsigned)B, (unsigned)((rows + threads - 1) / threads));
        if (arith == 2)
            ingest_u8_s2d44_kernel<2><<<grid, threads, 0, st>>>(obs, lut, (uint4 *)out, B, H, W, mul, add);
        else if (arith == 1)
            ingest_u8_s2d44_kernel<1><<<grid, threads, 0, st>>>(obs, lut, (uint4 *)out, B, H, W, mul, add);
        else
            ingest_u8_s2d44_kernel<0><<<grid, threads, 0, st>>>(obs, lut, (uint4 *)out, B, H, W, mul, add);
    } else {
        long long total = (long long)B * C * H * W;
        ingest_u8_s2d_any_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(obs, lut, out, total,
                                                                                 C, H, W, s);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// exhaustive verification of the fast division for one output scale
// ---------------------------------------------------------------------------------------
template <bool RELU>
__global__ void verify_fastdiv_kernel(float s, float r, float y_max, unsigned long long *bad)
{
    const unsigned long long total = 1ULL << 32;
    unsigned long long mine = 0;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (unsigned long long)gridDim.x * blockDim.x) {
        const float y = __uint_as_float((unsigned)i);
        if (!(fabsf(y) <= y_max)) continue;  // also skips NaN
        if (fastdiv_code<RELU>(y, s, r) != exact_code(y, s, RELU)) ++mine;
    }
    if (mine) atomicAdd(bad, mine);
}

// Compares fastdiv_code with the defining expression for every float |y| <= y_max.  Results are
// remembered per (scale, relu, range) so that a scale is checked once per process.
accerl_status verify_fastdiv(float s_out, float inv_s_out, bool relu, float y_max, bool *ok)
{
    struct Key {
        float s, r, ymax;
        bool relu, ok;
    };
    static std::vector<Key> cache;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    for (const Key &k : cache)
        if (k.s == s_out && k.r == inv_s_out && k.relu == relu && k.ymax >= y_max) {
            *ok = k.ok;
            return ACCERL_OK;
        }
    *ok = false;
    unsigned long long *bad = nullptr, host = 1;
    ACCERL_CUDA_TRY(cudaMalloc(&bad, sizeof(*bad)));
    cudaError_t e = cudaMemset(bad, 0, sizeof(*bad));
    if (e == cudaSuccess) {
        if (relu) verify_fastdiv_kernel<true><<<148 * 8, 256>>>(s_out, inv_s_out, y_max, bad);
        else verify_fastdiv_kernel<false><<<148 * 8, 256>>>(s_out, inv_s_out, y_max, bad);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpy(&host, bad, sizeof(host), cudaMemcpyDeviceToHost);
    cudaFree(bad);
    if (e != cudaSuccess) {
        set_error("verify_fastdiv: %s", cudaGetErrorString(e));
        return ACCERL_ERR_CUDA;
    }
    *ok = host == 0;
    cache.push_back(Key{s_out, inv_s_out, y_max, relu, *ok});
    return ACCERL_OK;
}

// Reciprocal for the three-step division by s_out: fl(1 / s_out) or, where that one fails the
// exhaustive comparison, one of its two neighbours (the correction step works with any reciprocal
// that close; which rare operand patterns round wrongly differs between them).  *fast_div = 0 and
// *inv_s_out = fl(1 / s_out) when none verifies or `allow` is false: the layer then runs the
// epilogue with the exact fallback near ties, which assumes the correctly rounded reciprocal.
accerl_status choose_fastdiv(float s_out, bool relu, float y_max, bool allow, float *inv_s_out, int *fast_div)
{
    volatile float inv = 1.0f / s_out;  // IEEE reciprocal, rounded once
    const float r0 = inv;
    *inv_s_out = r0;
    *fast_div = 0;
    if (!allow) return ACCERL_OK;
    const float cand[3] = {r0, nextafterf(r0, 2.f * r0), nextafterf(r0, 0.f)};
    for (float r : cand) {
        bool ok = false;
        accerl_status st = verify_fastdiv(s_out, r, relu, y_max, &ok);
        if (st != ACCERL_OK) return st;
        if (ok) {
            *inv_s_out = r;
            *fast_div = 1;
            return ACCERL_OK;
        }
    }
    return ACCERL_OK;
}

// ---------------------------------------------------------------------------------------
// plan
// ---------------------------------------------------------------------------------------

namespace {

bool conv_fits(const accerl_layer_desc &d)
{
    if (d.pad != 0 || d.kh % d.stride || d.in_h % d.stride || d.in_w % d.stride) return false;
    const int cs = d.stride * d.stride * d.in_c;
    if (cs != 32 && cs != 64 && cs != 128) return false;
    const int t = d.kh / d.stride;
    if (t * t > kTcMaxChunks) return false;
    if (d.out_c % 16 || d.out_c > 256) return false;
    if (d.stride != 1 && d.stride != 2 && d.stride != 4) return false;
    if (d.skip_from >= 0) return false;
    return true;
}

}  // namespace

accerl_status build_tc_plan(accerl_policy *p, const accerl_layer_desc *layers, int n_layers,
                            bool *used)
{
    *used = false;
    if (p->in_kind != ACCERL_IN_U8_NCHW || layers[0].kind != ACCERL_CONV2D) return ACCERL_OK;
    // ---- does every layer qualify?
    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        const LayerPlan &L = p->layers[i];
        const bool relu_in_noop = i > 0 && (layers[i - 1].flags & ACCERL_RELU_OUT);
        if ((d.flags & ACCERL_RELU_IN) && !relu_in_noop) return ACCERL_OK;
        if (d.kind == ACCERL_CONV2D) {
            if (!conv_fits(d)) return ACCERL_OK;
        } else if (d.kind == ACCERL_FC && fc_sample_fits(p, layers, n_layers, i)) {
            // runs fused with the sampler, whatever its size
        } else if (d.kind == ACCERL_FC) {
            const int K = L.in_h * L.in_w * L.in_cp;
            if (L.in_cp != L.in_c || K % 16 || K < 128 || (K + 127) / 128 > kTcMaxChunks)
                return ACCERL_OK;
            if (d.flags & ACCERL_LOGITS) {
                if (d.out_c > 256) return ACCERL_OK;
            } else if (d.out_c % 16 || d.out_c > kTcMaxN || (d.out_c > 256 && d.out_c % 256)) {
                return ACCERL_OK;
            }
        } else {
            return ACCERL_OK;
        }
    }
    for (int i = 0; i < n_layers; ++i)
        if ((long long)p->max_batch * p->layers[i].in_h * p->layers[i].in_w + 256 >= (1LL << 31))
            return ACCERL_OK;  // GEMM row indices are 32-bit
    // ---- layouts: a tensor is stored space-to-depth(s) when its reader is a conv of stride s
    for (int i = 0; i < n_layers; ++i)
        p->tensor_s2d[i] = layers[i].kind == ACCERL_CONV2D ? layers[i].stride : 1;
    p->tensor_s2d[n_layers] = 1;

    std::vector<Step> steps;
    bool fused_sample = false;
    Step s0;
    s0.kind = Step::INGEST_S2D;
    s0.kernel = (p->in_c == 4 && p->tensor_s2d[0] == 4) ? "ingest_u8_s2d44_kernel"
                                                        : "ingest_u8_s2d_any_kernel";
    s0.covers = "ingest";
    steps.push_back(s0);

    for (int i = 0; i < n_layers; ++i) {
        const accerl_layer_desc &d = layers[i];
        const LayerPlan &L = p->layers[i];
        if (fc_sample_fits(p, layers, n_layers, i)) {  // the last layer runs fused with the sampler
            Step fs;
            accerl_status fst = build_fc_sample(p, d, i, p->bufs[L.in_buf].ptr, L.in_c, &fs);
            if (fst != ACCERL_OK) return fst;
            steps.push_back(fs);
            fused_sample = true;
            continue;
        }
        TcStep ts;
        memset(&ts.prm, 0, sizeof(ts.prm));
        TcGemmParams &g = ts.prm;
        g.sub = 1;
        g.max_sub = 1;
        g.out_xmul = g.out2_xmul = 1;
        const bool logits = (d.flags & ACCERL_LOGITS) != 0;
        const int n_total = round_up(d.out_c, 16);
        g.n_total = n_total;
        g.n_tile = n_total > 256 ? 256 : n_total;
        if (d.kind == ACCERL_FC && !logits) {
            // small batches: narrower tiles, so that the weight stream is shared by more SMs
            const int m_tiles = (p->max_batch + 127) / 128;
            while (g.n_tile > 32 && g.n_tile % 32 == 0 && 2 * m_tiles * (n_total / g.n_tile) <= p->sm_count)
                g.n_tile /= 2;
        }
        g.n_tiles = n_total / g.n_tile;
        int rows_in_per_image, row_bytes;
        std::vector<int8_t> packed;
        if (d.kind == ACCERL_CONV2D) {
            const int s = d.stride, t = d.kh / s, Hs = d.in_h / s, Ws = d.in_w / s;
            const int CH = s * s * d.in_c;
            g.chunk_bytes = CH;
            g.n_chunks = t * t;
            rows_in_per_image = Hs * Ws;
            row_bytes = CH;
            g.rows_per_image = Hs * Ws;
            g.grid_w = Ws;
            g.shifted = 1;
            g.max_sub = 4;
            g.a_rows = round_up(128 + (t - 1) * Ws + (t - 1), 8);
            packed.assign((size_t)g.n_chunks * n_total * CH, 0);
            for (int by = 0; by < t; ++by)
                for (int bx = 0; bx < t; ++bx) {
                    const int j = by * t + bx;
                    g.row_off[j] = by * Ws + bx;
                    g.col_off[j] = 0;
                    for (int oc = 0; oc < d.out_c; ++oc)
                        for (int dy = 0; dy < s; ++dy)
                            for (int dx = 0; dx < s; ++dx)
                                for (int c = 0; c < d.in_c; ++c)
                                    packed[((size_t)j * n_total + oc) * CH + (dy * s + dx) * d.in_c + c] =
                                        d.w[((oc * d.in_c + c) * d.kh + s * by + dy) * d.kw + s * bx + dx];
                }
        } else {
            const int K = L.in_h * L.in_w * L.in_cp;
            g.chunk_bytes = 128;
            g.n_chunks = (K + 127) / 128;
            rows_in_per_image = 1;
            row_bytes = K;
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
        }
        g.out_h = L.out_h;
        g.out_w = L.out_w;
        const int so = p->tensor_s2d[i + 1];
        g.out_s2d = so;
        g.out_s2d_log2 = so == 4 ? 2 : (so == 2 ? 1 : 0);
        g.inv_rows_per_image = 1.0f / (float)g.rows_per_image;
        g.grid_w_magic = g.grid_w == 1 ? 0xffffffffu : (unsigned)(((1ULL << 32) + g.grid_w - 1) / g.grid_w);
        g.out_rows_per_image = (L.out_h / so) * (L.out_w / so);
        g.out_grid_w = L.out_w / so;
        g.out_pitch = so * so * n_total;
        g.kscale = L.kscale;
        g.bias = L.bias;
        g.s_out = L.s_out;
        g.relu_out = (d.flags & ACCERL_RELU_OUT) != 0;
        {
            volatile float inv = 1.0f / L.s_out;  // IEEE reciprocal, rounded once
            g.inv_s_out = inv;
        }
        const bool allow_fastdiv = !(p->flags & ACCERL_FLAG_TEST_NO_FASTDIV);
        // The single-fma requantiser where every channel has verified constants (searched first: a
        // layer that has them needs no check of the three-step division, 4.5 ms per output scale).
        std::vector<float> k_use(n_total, 0.f), b_use(n_total, 0.f);
        for (int c = 0; c < d.out_c; ++c) {
            volatile float k = d.s_in * d.s_w[c];  // one fp32 rounding, never contracted
            k_use[c] = k;
            b_use[c] = d.bias[c];
        }
        if (!logits && allow_fastdiv && !(p->flags & ACCERL_FLAG_TEST_NO_AFFINE)) {
            bool ok = false;
            std::vector<float> k2, b2;
            accerl_status vs = fit_affine_requant(k_use.data(), b_use.data(), n_total, g.s_out, g.relu_out != 0,
                                                  &k2, &b2, &ok);
            if (vs != ACCERL_OK) return vs;
            if (ok) {
                void *kd = nullptr, *bd = nullptr;
                if ((vs = upload_bytes(p, k2.data(), k2.size() * 4, &kd)) != ACCERL_OK) return vs;
                if ((vs = upload_bytes(p, b2.data(), b2.size() * 4, &bd)) != ACCERL_OK) return vs;
                g.kscale = (const float *)kd;
                g.bias = (const float *)bd;
                g.affine = 1;
                g.fast_div = 1;  // a verified division-free requantiser exists
                k_use = k2;
                b_use = b2;
            }
        }
        if (!logits && !g.affine) {
            // largest |y| = |fma(acc, k, b)| the layer can produce: |acc| < 2^31
            float kmax = 0.f, bmax = 0.f;
            for (int c = 0; c < d.out_c; ++c) {
                kmax = std::max(kmax, d.s_in * d.s_w[c]);
                bmax = std::max(bmax, fabsf(d.bias[c]));
            }
            accerl_status vs = choose_fastdiv(g.s_out, g.relu_out != 0, 2147483648.0f * kmax + bmax,
                                              allow_fastdiv, &g.inv_s_out, &g.fast_div);
            if (vs != ACCERL_OK) return vs;
        }
        const char *requant_note = g.affine ? "[single-fma requantiser verified]" : "[3-step divide verified]";
        g.split_cols = g.n_tile >= 128 ? 1 : 0;  // 128 / 256 columns: 32 / 64 per warpgroup
        g.out = L.out_buf >= 0 ? p->bufs[L.out_buf].ptr : nullptr;
        g.logits_mode = logits ? 1 : 0;
        g.n_actions = p->n_out;  // columns of the fp32 rows the logits layer writes
        g.status = p->status_word;
        g.trace_slot = (int)p->tc_steps.size();
        // resident weights when the whole matrix fits beside a useful pipeline
        ts.resident_b = g.n_tiles == 1 && (size_t)g.n_chunks * n_total * g.chunk_bytes <= 96 * 1024;
        if (g.shifted && (!ts.resident_b || g.a_rows > 256)) {
            g.shifted = 0;  // fall back to one box per tap
            g.a_rows = 128;
        }
        // The input stage runs inside the first conv when the frames have the shape the fused
        // producer is written for (4 channels, space-to-depth 4, 16-byte aligned strips) and the
        // quantiser is the fixed-point line; the parity tap of the quantised input needs the
        // separate launch.
        const bool fuse = i == 0 && d.kind == ACCERL_CONV2D && !unfuse_for_taps(p) &&
                          p->in_c == 4 && d.stride == 4 && g.chunk_bytes == 64 && g.shifted && ts.resident_b &&
                          p->ingest_arith == 1 && p->in_w % 4 == 0 && (p->in_h * p->in_w) % 16 == 0 && n_layers > 1;
        if (fuse) {
            TcGemmParams f = g;
            f.fuse_ingest = 1;
            f.max_sub = 2;
            f.in_w = p->in_w;
            f.in_plane = p->in_h * p->in_w;
            f.raw_rows = (f.grid_w - 1 + 128 + f.a_rows - 1) / f.grid_w + 1;  // two tiles per step
            f.ingest_mul = p->ingest_mul;
            f.ingest_add = p->ingest_add;
            f.ingest_clamp = 0;
            for (unsigned u = 0; u < 256; ++u)
                if (((unsigned long long)u * p->ingest_mul + p->ingest_add) >> 24 > 127) f.ingest_clamp = 1;
            if (p->ingest_shift1) f.ingest_clamp = 2;
            f.fuse_ingest = 0;  // the ordinary pipeline first: tiles per step, accumulators, issuing warps
            if (tc_choose_pipeline(f, true)) {
                f.fuse_ingest = 1;
                f.n_stages = f.n_mma;  // one stage per ring; the freed room holds the raw strips
                f.raw_rows = (f.grid_w - 1 + (f.sub - 1) * 128 + f.a_rows - 1) / f.grid_w + 1;
                if (tc_smem_bytes(f, true) <= 216 * 1024) g = f;
            }
        }
        // The dedicated first-conv kernel (tc_conv1.cu) takes the layer when it has the Atari shape:
        // 8 x 8 window, stride 4, 16 or 32 output channels, the verified division.
        if (fuse && g.fast_div) {
            Conv1Params c1;
            const int mode = p->ingest_shift1 ? 2 : (g.ingest_clamp ? 1 : 0);
            if (conv1_plan(d, p->in_h, p->in_w, p->max_batch, n_total, mode, &c1) &&
                conv1_smem_bytes(c1) <= 200 * 1024) {
                c1.ingest_mul = p->ingest_mul;
                c1.ingest_add = p->ingest_add;
                c1.out = g.out;
                c1.out_h = g.out_h;
                c1.out_w = g.out_w;
                c1.out_s2d_log2 = g.out_s2d_log2;
                c1.out_rows_per_image = g.out_rows_per_image;
                c1.out_grid_w = g.out_grid_w;
                c1.out_pitch = g.out_pitch;
                c1.n_total = n_total;
                c1.s_out = g.s_out;
                c1.inv_s_out = g.inv_s_out;
                c1.relu = g.relu_out;
                c1.affine = g.affine;
                c1.status = p->status_word;
                for (int c = 0; c < n_total; ++c) {
                    c1.ks[c] = k_use[c];
                    c1.bs[c] = b_use[c];
                }
                // weights [tap][channel][64 bytes], K ordered (c, dy, dx) as the bytes lie in the frame
                std::vector<int8_t> w1((size_t)4 * n_total * 64, 0);
                for (int by = 0; by < 2; ++by)
                    for (int bx = 0; bx < 2; ++bx)
                        for (int oc = 0; oc < d.out_c; ++oc)
                            for (int c = 0; c < 4; ++c)
                                for (int dy = 0; dy < 4; ++dy)
                                    for (int dx = 0; dx < 4; ++dx)
                                        w1[((size_t)(by * 2 + bx) * n_total + oc) * 64 + c * 16 + dy * 4 + dx] =
                                            d.w[((oc * 4 + c) * 8 + 4 * by + dy) * 8 + 4 * bx + dx];
                void *w1_dev = nullptr;
                accerl_status st1 = upload_bytes(p, w1.data(), w1.size(), &w1_dev);
                if (st1 != ACCERL_OK) return st1;
                st1 = tc_make_map(p->conv1_map_b, w1_dev, 4LL * n_total, 64, 64, n_total, 64);
                if (st1 != ACCERL_OK) return st1;
                p->conv1 = c1;
                Step s;
                s.kind = Step::CONV1_FRAMES;
                s.layer = i;
                s.kernel = std::string("conv1_frames_kernel") + requant_note + "[frames quantised inside]";
                s.covers = "ingest+layer 0";
                steps.clear();
                p->tap_missing[0] = 1;  // no quantised input tensor exists
                steps.push_back(s);
                continue;
            }
        }
        // Other strided convs on small grids with 48 or 64 output channels: the kernel with tiles of
        // whole grid rows (tc_conv.cu); the un-fused tap plan keeps the general kernel as cross-check.
        // (Measured at batch 8192: 64 channels 42.0 -> 36.5 and 37.9 -> 35.8 us for the second and
        // third layer; with 32 channels the general kernel is as fast or faster, 26.6 against 28.7 us.)
        if (d.kind == ACCERL_CONV2D && i > 0 && g.shifted && ts.resident_b && g.fast_div && !unfuse_for_taps(p) &&
            n_total > 32 && n_total <= 64) {
            ConvRowsStep cs;
            if (conv_rows_plan(g.rows_per_image / g.grid_w, g.grid_w, g.chunk_bytes, d.kh / d.stride, n_total,
                               p->max_batch, &cs.prm)) {
                ConvRowsParams &c2 = cs.prm;
                c2.out = g.out;
                c2.out_h = g.out_h;
                c2.out_w = g.out_w;
                c2.out_s2d_log2 = g.out_s2d_log2;
                c2.out_rows_per_image = g.out_rows_per_image;
                c2.out_grid_w = g.out_grid_w;
                c2.out_pitch = g.out_pitch;
                c2.n_total = n_total;
                c2.s_out = g.s_out;
                c2.inv_s_out = g.inv_s_out;
                c2.relu = g.relu_out;
                c2.affine = g.affine;
                c2.status = p->status_word;
                for (int c = 0; c < d.out_c; ++c) {
                    c2.ks[c] = k_use[c];
                    c2.bs[c] = b_use[c];
                }
                void *w2_dev = nullptr;
                accerl_status st2 = upload_bytes(p, packed.data(), packed.size(), &w2_dev);
                if (st2 != ACCERL_OK) return st2;
                st2 = tc_make_map(cs.map_a, p->bufs[L.in_buf].ptr, (long long)p->max_batch * rows_in_per_image,
                                  row_bytes, row_bytes, c2.box_rows, row_bytes);
                if (st2 != ACCERL_OK) return st2;
                st2 = tc_make_map(cs.map_b, w2_dev, (long long)g.n_chunks * n_total, row_bytes, row_bytes, n_total,
                                  row_bytes);
                if (st2 != ACCERL_OK) return st2;
                p->conv_rows.push_back(cs);
                Step s;
                s.kind = Step::CONV_ROWS;
                s.layer = i;
                s.tc = (int)p->conv_rows.size() - 1;
                s.kernel = std::string("conv_rows_kernel") + requant_note;
                s.covers = "layer " + std::to_string(i);
                steps.push_back(s);
                continue;
            }
        }
        if (!g.fuse_ingest && !tc_choose_pipeline(g, ts.resident_b)) {
            ts.resident_b = false;
            g.shifted = 0;
            g.a_rows = 128;
            if (!tc_choose_pipeline(g, false)) {  // generic plan stays
                p->tensor_s2d.assign(n_layers + 1, 1);
                p->tap_missing.assign(n_layers + 1, 0);
                p->tc_steps.clear();
                p->conv_rows.clear();
                return ACCERL_OK;
            }
        }
        void *w_dev = nullptr;
        accerl_status st = upload_bytes(p, packed.data(), packed.size(), &w_dev);
        if (st != ACCERL_OK) return st;
        const long long rows = (long long)p->max_batch * rows_in_per_image;
        st = tc_make_map(ts.map_a, p->bufs[L.in_buf].ptr, rows, row_bytes, row_bytes,
                         g.shifted ? g.a_rows : 128, g.chunk_bytes);
        if (st != ACCERL_OK) return st;
        st = tc_make_map(ts.map_b, w_dev, (long long)g.n_chunks * n_total, g.chunk_bytes,
                         g.chunk_bytes, g.n_tile, g.chunk_bytes);
        if (st != ACCERL_OK) return st;
        p->tc_steps.push_back(ts);
        Step s;
        s.kind = Step::TC_GEMM;
        s.layer = i;
        s.tc = (int)p->tc_steps.size() - 1;
        s.kernel = ts.resident_b ? "tc_gemm_kernel<resident weights>" : "tc_gemm_kernel<streamed weights>";
        if (g.fast_div) s.kernel += requant_note;
        else if (!logits) s.kernel += "[division check failed: exact divide near ties]";
        s.covers = "layer " + std::to_string(i);
        if (g.fuse_ingest) {  // takes the place of the ingest launch
            s.kernel += "[frames quantised inside]";
            s.covers = "ingest+layer 0";
            steps.clear();
            p->tap_missing[0] = 1;  // no quantised input tensor exists
        }
        steps.push_back(s);
    }
    if (!fused_sample) {
        Step ss;
        ss.kind = Step::SAMPLE;
        ss.kernel = p->n_actions <= 32 ? "sample_warp_kernel" : "sample_wide_kernel";
        ss.covers = "sample";
        steps.push_back(ss);
    }
    p->steps = steps;
    *used = true;
    return ACCERL_OK;
}

}  // namespace accerl
