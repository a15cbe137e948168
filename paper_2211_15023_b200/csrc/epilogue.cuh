// The fixed per-element arithmetic of the path, shared by every kernel of the library:
// input quantisation, the epilogue float and the requantisation.  Explicit round-to-nearest
// intrinsics keep the compiler from contracting or approximating anything.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace accerl {

// q = clamp(rintf(t), -128, 127) for a float that is already y / s
__device__ __forceinline__ int clamp_round_i8(float t)
{
    t = rintf(t);
    t = fminf(fmaxf(t, -128.f), 127.f);
    return (int)t;
}

// vector observation -> int8
__device__ __forceinline__ int8_t quantise_input(float x, float s_input)
{
    return (int8_t)clamp_round_i8(__fdiv_rn(x, s_input));
}

// y = fmaf((float)acc, k, b), ReLU if asked
__device__ __forceinline__ float epilogue_float(int acc, float k, float b, bool relu)
{
    float y = __fmaf_rn(__int2float_rn(acc), k, b);
    return relu ? fmaxf(y, 0.f) : y;
}

// q = clamp(rintf(y / s_out), -128, 127) with the IEEE divide
__device__ __forceinline__ int8_t requant(float y, float s_out)
{
    return (int8_t)clamp_round_i8(__fdiv_rn(y, s_out));
}

// Sixteen accumulators of one output position -> sixteen int8 codes in four words.
//
// Straight-line fast path: t = y * fl(1/s_out) differs from the IEEE quotient fl(y / s_out) by at
// most 1.5 * 2^-23 * |t| (one rounding in the reciprocal, one in the product, half an ulp in the
// quotient), i.e. by less than 2.4e-5 wherever the result is not clamped anyway (|t| <= 129).  So
// whenever t is farther than kTieGuard from a half-integer, rint(t) equals rint of the quotient;
// otherwise the element is redone with the exact divide.  Saturating conversion and saturating
// packing implement the clamp to [-128, 127].
constexpr float kTieGuard = 4e-5f;
constexpr float kRoundMagic = 12582912.f;  // 1.5 * 2^23: adding it rounds to the nearest integer

__device__ __forceinline__ uint32_t pack4_sat_s8(int a0, int a1, int a2, int a3)
{
    uint32_t hi, w;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi) : "r"(a3), "r"(a2));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(a1), "r"(a0), "r"(hi));
    return w;
}

__device__ __forceinline__ void requant16(const int (&acc)[16], const float (&ks)[16],
                                          const float (&bs)[16], bool relu, float s_out,
                                          float inv_s_out, uint32_t (&w)[4])
{
    int q[16];
    float worst = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float y = epilogue_float(acc[i], ks[i], bs[i], relu);
        const float t = __fmul_rn(y, inv_s_out);
        q[i] = __float2int_rn(t);
        worst = fmaxf(worst, fabsf(__fsub_rn(t, __int2float_rn(q[i]))));
    }
    if (worst > 0.5f - kTieGuard) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float y = epilogue_float(acc[i], ks[i], bs[i], relu);
            const float t = __fmul_rn(y, inv_s_out);
            if (fabsf(__fsub_rn(t, __int2float_rn(q[i]))) > 0.5f - kTieGuard)
                q[i] = __float2int_rn(__fdiv_rn(y, s_out));
        }
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) w[g] = pack4_sat_s8(q[4 * g], q[4 * g + 1], q[4 * g + 2], q[4 * g + 3]);
}

// max(code, 0) on four signed bytes: a byte permute in its sign-replicating mode gives 0xff for
// every negative byte, and those bytes are cleared
__device__ __forceinline__ uint32_t relu_bytes(uint32_t w)
{
    uint32_t neg;
    asm("prmt.b32 %0, %1, %1, 0xba98;" : "=r"(neg) : "r"(w));
    return w & ~neg;
}

// One requantised code by the three-step division: t = y * r, e = y - s * t (exact in one fma),
// d = t + e * r.  With r = fl(1 / s) this is the classical correctly rounded quotient except for
// rare operand patterns, so it is only used for scales for which fastdiv_code() has been compared
// with exact_code() over every fp32 value y can take (see verify_fastdiv in tc_plan.cu).  ReLU
// is applied to the code, which has the sign of y; the saturating pack does the clamp.
__device__ __forceinline__ int fastdiv_rint(float y, float s, float r)
{
    const float t = __fmul_rn(y, r);
    const float e = __fmaf_rn(-s, t, y);
    return __float2int_rn(__fmaf_rn(e, r, t));
}

// the defining expression, for one element: clamp(rintf(max?(y) / s), -128, 127)
__device__ __forceinline__ int exact_code(float y, float s, bool relu)
{
    if (relu) y = fmaxf(y, 0.f);
    return (int)requant(y, s);
}

template <bool RELU>
__device__ __forceinline__ int fastdiv_code(float y, float s, float r)
{
    const int q = min(max(fastdiv_rint(y, s, r), -128), 127);  // what the saturating pack does
    return RELU ? max(q, 0) : q;                               // and relu_bytes()
}

// Sixteen codes by the three-step division, two elements per instruction: the packed fp32
// operations of sm_100 round each half exactly as their scalar forms do, so the codes are those
// of fastdiv_code(); they only take half the issue slots.
template <bool RELU>
__device__ __forceinline__ void requant16_fastdiv(const int (&acc)[16], const float (&ks)[16],
                                                  const float (&bs)[16], float s_out,
                                                  float inv_s_out, uint32_t (&w)[4])
{
    int q[16];
    const float2 r2 = make_float2(inv_s_out, inv_s_out), ns2 = make_float2(-s_out, -s_out);
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const float2 a = make_float2(__int2float_rn(acc[i]), __int2float_rn(acc[i + 1]));
        const float2 y = __ffma2_rn(a, make_float2(ks[i], ks[i + 1]), make_float2(bs[i], bs[i + 1]));
        const float2 t = __fmul2_rn(y, r2);
        const float2 e = __ffma2_rn(ns2, t, y);
        const float2 d = __ffma2_rn(e, r2, t);
        q[i] = __float2int_rn(d.x);
        q[i + 1] = __float2int_rn(d.y);
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        w[g] = pack4_sat_s8(q[4 * g], q[4 * g + 1], q[4 * g + 2], q[4 * g + 3]);
        if (RELU) w[g] = relu_bytes(w[g]);
    }
}

// One code by a single fma: q = clamp(rint(fmaf((float)acc, k2, b2))), ReLU on the code.  The
// requantiser is a non-decreasing step function of the INTEGER accumulator, and so is this one
// (k2 > 0); for every output channel the pair (k2, b2) near (k / s_out, b / s_out) is searched at
// create until the two functions agree on every accumulator between the two points where both
// saturate, which makes them equal on all of int32 (fit_affine_requant in requant_fit.cu).
template <bool RELU>
__device__ __forceinline__ int affine_code(int acc, float k2, float b2)
{
    const int q = min(max(__float2int_rn(__fmaf_rn(__int2float_rn(acc), k2, b2)), -128), 127);
    return RELU ? max(q, 0) : q;
}

// sixteen codes by the single fma, two elements per instruction
template <bool RELU>
__device__ __forceinline__ void requant16_affine(const int (&acc)[16], const float (&k2)[16],
                                                 const float (&b2)[16], uint32_t (&w)[4])
{
    int q[16];
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        const float2 a = make_float2(__int2float_rn(acc[i]), __int2float_rn(acc[i + 1]));
        const float2 t = __ffma2_rn(a, make_float2(k2[i], k2[i + 1]), make_float2(b2[i], b2[i + 1]));
        q[i] = __float2int_rn(t.x);
        q[i + 1] = __float2int_rn(t.y);
    }
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        w[g] = pack4_sat_s8(q[4 * g], q[4 * g + 1], q[4 * g + 2], q[4 * g + 3]);
        if (RELU) w[g] = relu_bytes(w[g]);
    }
}

// Four frame bytes (byte `dx` of the words p0..p3, one per channel plane) -> four int8 codes in one
// word, channel 0 in the low byte, by the fixed-point line q = min((u * mul + add) >> 24, 127).
template <bool CLAMP>
__device__ __forceinline__ uint32_t ingest_fixed_line4(uint32_t p0, uint32_t p1, uint32_t p2, uint32_t p3,
                                                       int dx, uint32_t mul, uint32_t add)
{
    const uint32_t sel = 0x4440u + (uint32_t)dx;  // byte dx, zero extended
    const uint32_t r0 = __byte_perm(p0, 0, sel) * mul + add, r1 = __byte_perm(p1, 0, sel) * mul + add;
    const uint32_t r2 = __byte_perm(p2, 0, sel) * mul + add, r3 = __byte_perm(p3, 0, sel) * mul + add;
    // top bytes of the four multiply-adds
    const uint32_t lo = __byte_perm(r0, r1, 0x0073), hi = __byte_perm(r2, r3, 0x0073);
    const uint32_t codes = __byte_perm(lo, hi, 0x5410);
    return CLAMP ? __vminu4(codes, 0x7f7f7f7fu) : codes;  // without: the host saw the line stay <= 127
}

// The table q(u) = u >> 1 (what the input quantiser is when s_input = 1/127, the scale max-abs
// calibration gives whenever a calibration frame contains a 255): four words of four bytes each
// (one per channel plane, bytes = 4 pixels) -> four words of (channel 0..3) codes per pixel.
// Halving is done on all four bytes of a word at once; the rest is a 4 x 4 byte transpose.
__device__ __forceinline__ uint4 ingest_shift_line16(uint32_t p0, uint32_t p1, uint32_t p2, uint32_t p3)
{
    p0 = (p0 >> 1) & 0x7f7f7f7fu;
    p1 = (p1 >> 1) & 0x7f7f7f7fu;
    p2 = (p2 >> 1) & 0x7f7f7f7fu;
    p3 = (p3 >> 1) & 0x7f7f7f7fu;
    const uint32_t a = __byte_perm(p0, p1, 0x5140), b = __byte_perm(p0, p1, 0x7362);  // c0 c1 of pixels 0,1 / 2,3
    const uint32_t c = __byte_perm(p2, p3, 0x5140), d = __byte_perm(p2, p3, 0x7362);  // c2 c3
    return make_uint4(__byte_perm(a, c, 0x5410), __byte_perm(a, c, 0x7632), __byte_perm(b, d, 0x5410),
                      __byte_perm(b, d, 0x7632));
}

// Four frame bytes (byte `dx` of the words p0..p3, one per channel plane) -> four int8 codes in one
// word, channel 0 in the low byte, without integer multiplies: a byte permute builds the float
// 128 + u/256 from byte u, two packed float operations map it onto 1.5 * 2^23 + code (rounded to
// nearest by the addition itself), and the codes are the low bytes of the bit patterns.  The two
// constants come from fit_ingest_float_line(), which has checked all 256 inputs on the host.
__device__ __forceinline__ uint32_t ingest_float_line4(uint32_t p0, uint32_t p1, uint32_t p2, uint32_t p3,
                                                       int dx, float A, float c1)
{
    const uint32_t sel = 0x7404u | ((uint32_t)dx << 4);  // bytes: 00, u, 00, 0x43
    const float2 f01 = make_float2(__uint_as_float(__byte_perm(p0, 0x43000000u, sel)),
                                   __uint_as_float(__byte_perm(p1, 0x43000000u, sel)));
    const float2 f23 = make_float2(__uint_as_float(__byte_perm(p2, 0x43000000u, sel)),
                                   __uint_as_float(__byte_perm(p3, 0x43000000u, sel)));
    const float2 nc = make_float2(-c1, -c1), a2 = make_float2(A, A), mg = make_float2(kRoundMagic, kRoundMagic);
    const float2 r01 = __ffma2_rn(__fadd2_rn(f01, nc), a2, mg);
    const float2 r23 = __ffma2_rn(__fadd2_rn(f23, nc), a2, mg);
    const uint32_t lo = __byte_perm(__float_as_uint(r01.x), __float_as_uint(r01.y), 0x0040);
    const uint32_t hi = __byte_perm(__float_as_uint(r23.x), __float_as_uint(r23.y), 0x0040);
    return __byte_perm(lo, hi, 0x5410);
}

}  // namespace accerl
