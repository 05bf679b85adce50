// Activation / weight quantization kernels (Sec. 3 uniform quantizer, Sec. 4.3.2 Q_dual and polarity
// split, Sec. 4.2.2 one scale per segment; App. A zero-point quantizer as a mode; the act-to-linear prologue of
// Sec. 4.3.2 compiled in on request; per-row scales and 4-bit packing for the W4A8 setting of App. B).
// HBM-streaming: every thread converts 16 consecutive elements per row (the row pieces arrive through a
// thread-private ring of asynchronous 16-byte copies in shared memory, one 128-bit store per code matrix goes out)
// and walks down the rows with that column chunk.  The codes are those of "one IEEE fp32 division, round half to
// even, clip"; the common case computes them with a handful of full-rate fp32 instructions per element (see
// SegConst) so that the pass stays memory bound.
#include <cuda_bf16.h>
#include <atomic>
#include "sq_common.cuh"

namespace sq {
namespace {

constexpr int kThreads = 256;
constexpr int kVec = 16;             // elements per thread and row
#ifndef SQ_QUANT_BLOCKS_PER_SM
#define SQ_QUANT_BLOCKS_PER_SM 4
#endif
constexpr int kBlocksPerSm = SQ_QUANT_BLOCKS_PER_SM;   // resident blocks per SM the kernel is compiled for (4: at most 64 registers)

// 16 consecutive elements of a row as loaded (fp32: four 128-bit words, bf16: two), converted when used
template <typename Tin> struct Raw16;
template <> struct Raw16<float> { float4 v[4]; };
template <> struct Raw16<__nv_bfloat16> { uint4 v[2]; };

__device__ __forceinline__ void load16(const float *p, Raw16<float> &r)
{
    const float4 *q = reinterpret_cast<const float4 *>(p);
#pragma unroll
    for (int i = 0; i < 4; i++) r.v[i] = __ldg(q + i);
}
__device__ __forceinline__ void load16(const __nv_bfloat16 *p, Raw16<__nv_bfloat16> &r)
{
    const uint4 *q = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int i = 0; i < 2; i++) r.v[i] = __ldg(q + i);
}
// piece v (16 bytes) of a row chunk
__device__ __forceinline__ void set_piece(Raw16<float> &r, int v, uint4 w)
{
    r.v[v] = make_float4(__uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z), __uint_as_float(w.w));
}
__device__ __forceinline__ void set_piece(Raw16<__nv_bfloat16> &r, int v, uint4 w) { r.v[v] = w; }

// elements 4 g .. 4 g + 3 as fp32
__device__ __forceinline__ void get4(const Raw16<float> &r, int g, float (&x)[4])
{
    x[0] = r.v[g].x; x[1] = r.v[g].y; x[2] = r.v[g].z; x[3] = r.v[g].w;
}
__device__ __forceinline__ void get4(const Raw16<__nv_bfloat16> &r, int g, float (&x)[4])
{
    const uint4 v = r.v[g >> 1];
    const uint32_t w0 = (g & 1) ? v.z : v.x, w1 = (g & 1) ? v.w : v.y;
    x[0] = __uint_as_float(w0 << 16); x[1] = __uint_as_float(w0 & 0xFFFF0000u);
    x[2] = __uint_as_float(w1 << 16); x[3] = __uint_as_float(w1 & 0xFFFF0000u);
}

__device__ __forceinline__ float load1(const float *p) { return __ldg(p); }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p)
{
    return __uint_as_float(uint32_t(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
}

// two fp32 -> two e4m3 bytes (round-to-nearest-even, saturate to +-448); low byte = a.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float a, float b)
{
    unsigned short r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(b), "f"(a));
    return r;
}

enum : int { kSingle = 0, kDual = 1, kZeroPoint = 2 };   // quantizer modes

// One element -> (code for the positive / only matrix, code for the negative matrix), as bytes.
// Reference form: one IEEE division, round half to even, clip.  Used where a vector straddles a
// segment bound or the end of a row, and for scales outside the range of the fast form below.
// Zero-point mode (App. A asymmetric quantizer): clip(round(x / s) + z, lo, hi), z passed in `zp`.
template <int CODE, int MODE>
__device__ __forceinline__ void quant1(float x, float sp, float sn, int zp, int lo, int hi, uint32_t &cp, uint32_t &cn)
{
    constexpr bool DUAL = MODE == kDual;
    if (CODE == SQ_CODE_INT8) {
        float s = DUAL ? (x >= 0.0f ? sp : sn) : sp;
        int c = __float2int_rn(__fdiv_rn(x, s));      // IEEE divide, round half to even, saturating convert
        if (MODE == kZeroPoint) c = max(min(c, 1000000), -1000000) + zp;
        c = max(min(c, hi), lo);
        if (DUAL) { cp = uint32_t(max(c, 0)) & 0xFFu; cn = uint32_t(min(c, 0)) & 0xFFu; }
        else      { cp = uint32_t(c) & 0xFFu; cn = 0; }
    } else {
        bool pos = x >= 0.0f;
        float s = DUAL ? (pos ? sp : sn) : sp;
        uint32_t c = cvt_e4m3x2(__fdiv_rn(x, s), 0.0f) & 0xFFu;
        if ((c & 0x7Fu) == 0) c = 0;                  // -0 is stored as +0
        if (DUAL) { cp = pos ? c : 0u; cn = pos ? 0u : c; }
        else      { cp = c; cn = 0; }
    }
}

// The act-to-linear segment in front of the quantizer (Sec. 4.3.2; App. B: SiLU and GELU feed DualScale layers),
// evaluated in fp32 and rounded once to the dtype the unfused graph would have stored the activation in.
// SiLU(h) = h sigma(h) with z = exp(-|h|): sigma = 1 / (1 + z) for h >= 0, z / (1 + z) below (no overflow).  The
// exponential is the hardware base-2 approximation of h log2(e) (the rounding of that product costs |h| 2^-24
// relative, the approximation itself about one unit in the last place) and the division the hardware's fast one
// (2 units in the last place for a divisor in [1, 2]): relative error <= (|h| + 8) 2^-23, a fraction of a bf16
// half-step (2^-9) for every |h| below the underflow of the result.
// GELU(h) = h Phi(h) with E = erfc(t), t = |h| / sqrt 2: h (1 - E / 2) for h >= 0, (h / 2) E below.
// erfc(t) = exp(-t^2) g(t); the smooth factor g (the scaled complementary error function) is a degree-9
// polynomial in z = (t - 2.5) / (t + 2.5), which maps [0, 9.6] into [-1, 0.59) (coefficients from a least-squares
// fit of the relative error on Chebyshev nodes, 2^-29, by gelu_coefficients.py; beyond t = 9.6 the exponential
// has underflowed).  t^2 is
// split into its rounded value s and the rounding error e = fma(t, t, -s), and exp(-t^2) = exp(-s) (1 - e) to
// first order, so that the rounding of the square, which the exponential would amplify by t^2, does not count.
// What remains is the hardware exponential's own error (|s| 2^-24 from the product with log2 e, one unit in the
// last place from the approximation), the fast division's 2 units and a dozen roundings: relative error
// <= (3 h^2 + 48) 2^-24; in |h| <= 4 it stays below 2^-20.
__device__ __forceinline__ float silu_f32(float h)
{
    const float z = __expf(-fabsf(h));
    const float num = h >= 0.0f ? h : __fmul_rn(h, z);
    return __fdividef(num, __fadd_rn(1.0f, z));
}
__device__ __forceinline__ float gelu_f32(float h)
{
    const float t = __fmul_rn(fabsf(h), 0.70710678118654752440f);
    const float z = __fdividef(t - 2.5f, t + 2.5f);
    float g = -5.388610225e-05f;
    g = fmaf(g, z, 2.161547454e-04f);
    g = fmaf(g, z, 8.157527773e-04f);
    g = fmaf(g, z, -2.643950749e-03f);
    g = fmaf(g, z, -3.974915482e-03f);
    g = fmaf(g, z, 3.992317244e-02f);
    g = fmaf(g, z, -1.250353903e-01f);
    g = fmaf(g, z, 2.517131865e-01f);
    g = fmaf(g, z, -3.717366457e-01f);
    g = fmaf(g, z, 2.108063698e-01f);
    const float s = __fmul_rn(t, t);
    const float e = fmaf(t, t, -s);                       // t^2 = s + e exactly
    float E = __fmul_rn(__expf(-s), g);
    E = fmaf(-E, e, E);                                   // exp(-(s + e)) = exp(-s) (1 - e) to first order
    const float half = __fmul_rn(0.5f, h);
    const float v = h >= 0.0f ? fmaf(-half, E, h) : __fmul_rn(half, E);
    // beyond t = 13.5 the exponential has long underflowed: h or -0, also where t^2 overflows or h is infinite
    return t >= 13.5f ? (h >= 0.0f ? h : -0.0f) : v;
}
template <typename Tin>
__device__ __forceinline__ float pre1(float h, int act, float mult)
{
    float a = h;
    if (act) {
        a = act == 1 ? silu_f32(h) : gelu_f32(h);
        if (sizeof(Tin) == 2) a = __bfloat162float(__float2bfloat16_rn(a));      // stored as bf16 in the unfused graph
    }
    return __fmul_rn(a, mult);                                // the per-channel multiplier: one fp32 multiply
}
// Gated GELU (App. B lists GEGLU with SiLU and GELU): value * GELU(gate), the product in fp32 (one more rounding
// on top of the GELU's error: relative error <= (3 g^2 + 49) 2^-24), rounded once to the stored dtype.
template <typename Tin>
__device__ __forceinline__ float pre_gated(float value, float gate, float mult)
{
    float a = __fmul_rn(value, gelu_f32(gate));
    if (sizeof(Tin) == 2) a = __bfloat162float(__float2bfloat16_rn(a));
    return __fmul_rn(a, mult);
}

// Per-segment constants of the fast form.  The quotient x / s is obtained from the correctly rounded
// reciprocal r = RN(1/s) by one multiply and two FMAs,
//   q0 = RN(x r),  e = x - q0 s (exact in one FMA),  q = RN(q0 + e r),
// which lands on the same side of every rounding boundary of the codes (k + 1/2 for int8, the midpoints of
// adjacent e4m3 values) as RN(x / s), provided e is exact, i.e. does not underflow: |x| >= 2^-100 suffices, and for
// smaller |x| the quotient is below 2^-20 for the scales of the fast form (2^-80 <= s <= 2^100) and the code is 0
// whatever its last bits are.  (Checked on the CPU against the IEEE division for 2 * 10^10 inputs within six
// units in the last place of a rounding boundary, scales with random, all-ones and power-of-two significands.)
struct SegConst {
    float s, r;        // scale and RN(1 / s)
    float inv_l;       // e4m3 form: 1 / L with L = 2^(exponent(s) + 11) >= 1024 s
    float s_l, r_l;    // e4m3 form: s / L and RN(L / s)
    int fast;
};
__device__ __forceinline__ SegConst seg_const(float s)
{
    SegConst c;
    c.fast = (s >= 8.2718061255302767e-25f && s <= 1.2676506002282294e+30f) ? 1 : 0;     // 2^-80 .. 2^100
    c.s = s;
    c.r = __frcp_rn(s);
    const uint32_t l_bits = (__float_as_uint(s) & 0x7F800000u) + (11u << 23);
    const float l = __uint_as_float(l_bits);
    c.inv_l = __uint_as_float((254u << 23) - l_bits);
    c.s_l = s * c.inv_l;
    c.r_l = c.r * l;
    return c;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c)
{
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// packed fp32 pairs: sm_100 executes mul / fma / add on two fp32 values per instruction
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void unpack2u(uint64_t v, uint32_t &lo, uint32_t &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// two quotients x / s from r = RN(1/s): q0 = RN(x r), e = x - q0 s, q = RN(q0 + e r)
__device__ __forceinline__ uint64_t div2_rn_fast(uint64_t x2, uint64_t neg_s2, uint64_t r2)
{
    const uint64_t q0 = mul2(x2, r2);
    const uint64_t e = fma2(q0, neg_s2, x2);
    return fma2(e, r2, q0);
}
// {sat_s8(hi_val), sat_s8(lo_val)} into bits 15..0 of the result, bits 15..0 of `upper` into bits 31..16
__device__ __forceinline__ uint32_t pack_sat_s8(int hi_val, int lo_val, uint32_t upper)
{
    uint32_t d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(hi_val), "r"(lo_val), "r"(upper));
    return d;
}

constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23: v + magic rounds v to an integer, half to even
constexpr int kMagicBits = 0x4B400000;       // its bit pattern: bits(v + magic) - kMagicBits is that integer

// 4 elements of one K-segment -> one word of packed codes per matrix.
// int8, dual: both polarities are quantized as non-negative numbers, max(x, 0) and max(-x, 0) = max(x, 0) - x,
//   each with its own constants.  Adding the magic constant rounds half to even; the integer is the distance of
//   the sum's bit pattern from the constant's, taken with the sign of the polarity, and a saturating pack clips
//   it to [-128, 127].  A quotient beyond the range of the magic constant, infinity, or the NaN of an overflowed
//   chain all have bit patterns above the constant's, so they saturate to the end of the code range as the
//   clip demands; nothing has to be bounded beforehand.  (A negative bound of -127 takes the division path.)
// int8, single scale: |x| is quantized, clipped in fp32 (clip-then-round equals round-then-clip for integer
//   bounds; a NaN from an overflowed chain clips to the bound as well) and the sign put back when rounding.
// e4m3: the input is first mapped to u = sat(x / L) in [0, 1] with one saturating FMA (L a power of two, so
//   u / (s / L) has the bits of x / s; x beyond L is clipped to 448 anyway), which also splits the polarities and
//   keeps infinities and NaNs out of the saturating e4m3 conversion.
template <int CODE, int MODE>
__device__ __forceinline__ void quant4(const float (&x)[4], const SegConst &cp, const SegConst &cn, float hi, int zp,
                                       uint32_t &wp, uint32_t &wn)
{
    constexpr bool DUAL = MODE == kDual;
    const uint64_t magic2 = pack2(kRoundMagic, kRoundMagic);
    if (MODE == kZeroPoint) {
        // round(|x| / s) with the sign of x (the magnitude clipped at 256: anything beyond leaves the code range
        // whatever z is; a NaN from an overflowed chain clips the same way), plus z, saturated to [-128, 127]
        const uint64_t r2 = pack2(cp.r, cp.r), ns2 = pack2(-cp.s, -cp.s);
        const int off = zp - kMagicBits;
        int k[4];
#pragma unroll
        for (int i = 0; i < 4; i += 2) {
            float a0, a1;
            unpack2(div2_rn_fast(pack2(fabsf(x[i]), fabsf(x[i + 1])), ns2, r2), a0, a1);
            k[i] = int(__float_as_uint(fmaf(fminf(a0, 256.0f), copysignf(1.0f, x[i]), kRoundMagic))) + off;
            k[i + 1] = int(__float_as_uint(fmaf(fminf(a1, 256.0f), copysignf(1.0f, x[i + 1]), kRoundMagic))) + off;
        }
        wp = pack_sat_s8(k[1], k[0], pack_sat_s8(k[3], k[2], 0u));
        return;
    }
    if (CODE == SQ_CODE_INT8 && DUAL) {
        const uint64_t rp2 = pack2(cp.r, cp.r), nsp2 = pack2(-cp.s, -cp.s);
        const uint64_t rn2 = pack2(cn.r, cn.r), nsn2 = pack2(-cn.s, -cn.s);
        const uint64_t minus1 = pack2(-1.0f, -1.0f);
        int kp[4], kn[4];
#pragma unroll
        for (int i = 0; i < 4; i += 2) {
            const uint64_t xp2 = pack2(fmaxf(x[i], 0.0f), fmaxf(x[i + 1], 0.0f));
            const uint64_t xn2 = fma2(pack2(x[i], x[i + 1]), minus1, xp2);          // max(x, 0) - x, exact
            uint32_t a, b;
            unpack2u(add2(div2_rn_fast(xp2, nsp2, rp2), magic2), a, b);
            kp[i] = int(a) - kMagicBits; kp[i + 1] = int(b) - kMagicBits;
            unpack2u(add2(div2_rn_fast(xn2, nsn2, rn2), magic2), a, b);
            kn[i] = kMagicBits - int(a); kn[i + 1] = kMagicBits - int(b);
        }
        wp = pack_sat_s8(kp[1], kp[0], pack_sat_s8(kp[3], kp[2], 0u));
        wn = pack_sat_s8(kn[1], kn[0], pack_sat_s8(kn[3], kn[2], 0u));
        return;
    }
    uint32_t bp[4], bn[4];
    if (CODE == SQ_CODE_INT8) {                          // single scale
        const uint64_t r2 = pack2(cp.r, cp.r), ns2 = pack2(-cp.s, -cp.s);
#pragma unroll
        for (int i = 0; i < 4; i += 2) {
            float a0, a1;
            unpack2(div2_rn_fast(pack2(fabsf(x[i]), fabsf(x[i + 1])), ns2, r2), a0, a1);
            bp[i] = __float_as_uint(fmaf(fminf(a0, hi), copysignf(1.0f, x[i]), kRoundMagic));
            bp[i + 1] = __float_as_uint(fmaf(fminf(a1, hi), copysignf(1.0f, x[i + 1]), kRoundMagic));
        }
        wp = __byte_perm(__byte_perm(bp[0], bp[1], 0x0040), __byte_perm(bp[2], bp[3], 0x0040), 0x5410);
        return;
    }
    // e4m3
    const uint64_t rp2 = pack2(cp.r_l, cp.r_l), nsp2 = pack2(-cp.s_l, -cp.s_l);
    const uint64_t rn2 = pack2(cn.r_l, cn.r_l), nsn2 = pack2(-cn.s_l, -cn.s_l);
#pragma unroll
    for (int i = 0; i < 4; i += 2) {
        float a0, a1;
        if (DUAL) {
            unpack2(div2_rn_fast(pack2(fma_sat(x[i], cp.inv_l, 0.0f), fma_sat(x[i + 1], cp.inv_l, 0.0f)), nsp2, rp2), a0, a1);
            bp[i] = __float_as_uint(a0); bp[i + 1] = __float_as_uint(a1);
            unpack2(div2_rn_fast(pack2(fma_sat(x[i], -cn.inv_l, 0.0f), fma_sat(x[i + 1], -cn.inv_l, 0.0f)), nsn2, rn2), a0, a1);
            bn[i] = __float_as_uint(a0); bn[i + 1] = __float_as_uint(a1);
        } else {
            unpack2(div2_rn_fast(pack2(fma_sat(fabsf(x[i]), cp.inv_l, 0.0f), fma_sat(fabsf(x[i + 1]), cp.inv_l, 0.0f)), nsp2, rp2), a0, a1);
            bp[i] = __float_as_uint(copysignf(a0, x[i])); bp[i + 1] = __float_as_uint(copysignf(a1, x[i + 1]));
        }
    }
    uint32_t w = cvt_e4m3x2(__uint_as_float(bp[0]), __uint_as_float(bp[1])) |
                 (cvt_e4m3x2(__uint_as_float(bp[2]), __uint_as_float(bp[3])) << 16);
    // single scale: -0 is stored as +0; dual: the positive matrix holds non-negative quotients, no -0 arises
    wp = DUAL ? w : w & ~(__vcmpeq4(w & 0x7F7F7F7Fu, 0u) & 0x80808080u);
    if (DUAL) {
        // the negative matrix was quantized as magnitudes: set the sign bit of every nonzero byte
        // (a byte b <= 0x7E plus 0x7F reaches 0x80 exactly when b >= 1, and never carries into the next byte)
        w = cvt_e4m3x2(__uint_as_float(bn[0]), __uint_as_float(bn[1])) |
            (cvt_e4m3x2(__uint_as_float(bn[2]), __uint_as_float(bn[3])) << 16);
        wn = w | ((w + 0x7F7F7F7Fu) & 0x80808080u);
    }
}

// Thread g of the grid owns the 16-element column chunk g % V of the rows g / V, g / V + R, g / V + 2 R, ...
// (V chunks per row, R rows in flight over the whole grid), so that a warp reads 1 KiB (bf16) of consecutive
// addresses per row, the per-segment constants are made once per thread, and the next row's loads are in
// flight while the current row is converted.
// PRE != 0 compiles in the act-to-linear prologue: activation function and per-channel multiplier in front of the
// quantizer, so that the activation's output never goes through HBM.  PRE == 2 is the gated form: the row holds
// 2 K pre-activations, the value half travels through the ring like any input and the gate half (K elements
// further on) is fetched into registers one row ahead.
// RING: depth of the shared-memory ring the rows travel through (see below); 4 when a thread has many rows to
// walk (large inputs: more bytes in flight), 2 otherwise (less shared memory, more L1 for the copies).
template <typename Tin, int CODE, int MODE, int PRE, int RING>
__global__ void __launch_bounds__(kThreads, PRE ? 3 : kBlocksPerSm)
quantize_kernel(const __grid_constant__ QuantParams prm)
{
    constexpr bool DUAL = MODE == kDual;
    constexpr bool GATED = PRE == 2;
    // Programmatic dependent launch: this kernel may be scheduled while the previous kernel of the stream
    // winds down, and lets the next one be scheduled while its own last blocks run; nothing in global
    // memory is touched before the previous kernel has completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const SegBounds &sb = prm.sb;
    const int64_t M = prm.M;
    const int K = prm.K, R = prm.R, lo = prm.lo, hi = prm.hi, row_segments = prm.row_segments;
    const uint32_t g = blockIdx.x * kThreads + threadIdx.x;
    const uint32_t r0 = g / uint32_t(prm.V);
    if (r0 >= uint32_t(R) || int64_t(r0) >= M) return;
    const int k0 = int(g - r0 * uint32_t(prm.V)) * kVec;

    // K-segment of this chunk (bounds come with the kernel parameters)
    int p = 0;
    while (p + 1 < sb.P && k0 >= sb.kb[p + 1]) p++;
    const bool whole = k0 + kVec <= sb.kb[p + 1];            // chunk inside one K-segment (and inside K)
    const int Qs = row_segments ? sb.Q : 1;

    const Tin *src = static_cast<const Tin *>(prm.X) + int64_t(r0) * prm.ld + k0;
    uint8_t *dp = prm.c_pos + int64_t(r0) * prm.ldc + k0;
    uint8_t *dn = DUAL ? prm.c_neg + int64_t(r0) * prm.ldc + k0 : nullptr;
    const int64_t src_step = int64_t(R) * prm.ld, dst_step = int64_t(R) * prm.ldc;

    float mreg[PRE ? kVec : 1];                              // this chunk's multipliers, loaded once
    if (PRE) {
#pragma unroll
        for (int i = 0; i < kVec; i++) mreg[i] = (prm.mult && k0 + i < K) ? __ldg(prm.mult + k0 + i) : 1.0f;
    }

    // The rows of this chunk travel through a thread-private ring in shared memory: asynchronous 16-byte copies
    // (global -> shared without passing through registers) of the next kDepth - 1 rows are in flight while the
    // current row is converted, so the bytes in flight per SM do not cost registers.  Every thread reads only what
    // it copied itself, so a wait on its own copy groups is all the synchronisation there is.
    constexpr int NV = int(sizeof(Tin)) * kVec / 16;                        // 16-byte pieces per row chunk
    constexpr int kDepth = (sizeof(Tin) == 2 || RING == 2) ? RING : RING / 2;  // ring slots (32 KiB per block at most)
    __shared__ uint4 ring[kDepth * NV * kThreads];
    const uint32_t ring0 = uint32_t(__cvta_generic_to_shared(ring)) + threadIdx.x * 16u;
    auto slot_addr = [&](int slot, int v) { return ring0 + uint32_t((slot * NV + v) * kThreads) * 16u; };
    auto copy_row = [&](const Tin *row_src, int slot, bool valid) {          // one commit group per call, always
        if (valid) {
#pragma unroll
            for (int v = 0; v < NV; v++)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(slot_addr(slot, v)),
                             "l"(reinterpret_cast<const char *>(row_src) + 16 * v) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto read_row = [&](int slot, Raw16<Tin> &r) {
#pragma unroll
        for (int v = 0; v < NV; v++) {
            uint4 w;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w)
                         : "r"(slot_addr(slot, v)) : "memory");
            set_piece(r, v, w);
        }
    };
    if (whole) {
#pragma unroll
        for (int d = 0; d < kDepth - 1; d++) copy_row(src + int64_t(d) * src_step, d, int64_t(r0) + int64_t(d) * R < M);
    }
    const Tin *gsrc = src + K;                               // (gated) this chunk of the gate half
    Raw16<Tin> gate_next;
    if (GATED && whole) load16(gsrc, gate_next);
    int q = 0;                                               // N-segment (weights only) the constants belong to
    int64_t q_end = 0;                                       // first row beyond it (0: no constants yet)
    SegConst cp, cn;
    int zp = 0;
    bool fast = false;
    int slot = 0;                                            // ring slot of the current row
    for (int64_t row = r0; row < M; row += R) {
        if (row >= q_end) {                                  // (weights) the row entered another N-segment
            if (row_segments) {
                while (q + 1 < sb.Q && row >= sb.nb[q + 1]) q++;
                q_end = sb.nb[q + 1];
            } else {
                q_end = M;
            }
            cp = seg_const(__ldg(prm.s_pos + p * Qs + (row_segments ? q : 0)));
            cn = seg_const(DUAL ? __ldg(prm.s_neg + p * Qs + (row_segments ? q : 0)) : 1.0f);
            if (MODE == kZeroPoint) zp = __ldg(prm.zp + p);
            fast = whole && cp.fast && cn.fast && !(DUAL && CODE == SQ_CODE_INT8 && lo != -128);
        }
        Raw16<Tin> cur, gate;
        if (GATED && whole) {
            gate = gate_next;
            if (row + R < M) load16(gsrc + src_step, gate_next);
        }
        if (whole) {
            // row + (kDepth - 1) R goes into the slot the previous row has just left; then the oldest group, this
            // row's, is complete once at most kDepth - 1 newer groups are pending
            const int ahead = slot == 0 ? kDepth - 1 : slot - 1;
            copy_row(src + int64_t(kDepth - 1) * src_step, ahead, row + int64_t(kDepth - 1) * R < M);
            asm volatile("cp.async.wait_group %0;" ::"n"(kDepth - 1) : "memory");
            if (fast) read_row(slot, cur);
            slot = slot + 1 == kDepth ? 0 : slot + 1;
        }
        if (fast) {
            uint32_t wp[4], wn[4];
#pragma unroll
            for (int g4 = 0; g4 < 4; g4++) {
                float x[4];
                get4(cur, g4, x);
                if (GATED) {
                    float gt[4];
                    get4(gate, g4, gt);
#pragma unroll
                    for (int i = 0; i < 4; i++) x[i] = pre_gated<Tin>(x[i], gt[i], mreg[PRE ? 4 * g4 + i : 0]);
                } else if (PRE) {
#pragma unroll
                    for (int i = 0; i < 4; i++) x[i] = pre1<Tin>(x[i], prm.act, mreg[PRE ? 4 * g4 + i : 0]);
                }
                quant4<CODE, MODE>(x, cp, cn, float(hi), zp, wp[g4], wn[g4]);
            }
            *reinterpret_cast<uint4 *>(dp) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
            if (DUAL) *reinterpret_cast<uint4 *>(dn) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
        } else {                                 // segment bound or end of row inside the chunk, or an extreme scale
            const int n = min(kVec, K - k0);
            int pp = p;
            const int qq = row_segments ? q : 0;
            for (int i = 0; i < n; i++) {
                while (pp + 1 < sb.P && k0 + i >= sb.kb[pp + 1]) pp++;
                uint32_t a, b;
                float x = load1(src + i);
                if (GATED) x = pre_gated<Tin>(x, load1(gsrc + i), prm.mult ? __ldg(prm.mult + k0 + i) : 1.0f);
                else if (PRE) x = pre1<Tin>(x, prm.act, prm.mult ? __ldg(prm.mult + k0 + i) : 1.0f);
                quant1<CODE, MODE>(x, __ldg(prm.s_pos + pp * Qs + qq), DUAL ? __ldg(prm.s_neg + pp * Qs + qq) : 0.0f,
                                   MODE == kZeroPoint ? __ldg(prm.zp + pp) : 0, lo, hi, a, b);
                dp[i] = uint8_t(a);
                if (DUAL) dn[i] = uint8_t(b);
            }
        }
        src += src_step;
        if (GATED) gsrc += src_step;
        dp += dst_step;
        if (DUAL) dn += dst_step;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");     // nothing of this thread's is in flight when it leaves
}

// ----------------------------------------------------------------------------- fused activation by table (bf16 inputs)
// A bf16 pre-activation has 65536 possible values, so the stored activation bf16(act(h)) is a table of 128 KiB.
// Every CTA (1024 threads, one per SM) builds the table in its shared memory with the same silu_f32 / gelu_f32 as
// the arithmetic variant (a few evaluations per thread: most bit patterns need none), after which an element costs one
// shared-memory load instead of about 30 instructions: the fused pass stops being bound by the ALUs.  Results are
// those of the arithmetic variant bit for bit.  Used for large inputs: a launch of this kernel costs about 9 us
// more than the other's (the table, and a CTA that fills the SM cannot start under the previous kernel's tail).
// (Not for the gated form: its product is rounded once, from the unrounded GELU, which a bf16 table does not hold.)
// The rest is quantize_kernel's scheme: thread g owns column chunk g % V of rows g / V, g / V + R, ...; the rows
// travel through a thread-private ring of kTableDepth slots behind the table.
constexpr int kTableThreads = 1024;
constexpr int kTableDepth = 3;
constexpr size_t kTableBytes = 65536 * 2;
constexpr size_t kTableSmem = kTableBytes + size_t(kTableDepth) * 2 * kTableThreads * 16;      // 224 KiB

template <int CODE, int MODE>
__global__ void __launch_bounds__(kTableThreads, 1)
quantize_table_kernel(const __grid_constant__ QuantParams prm)
{
    constexpr bool DUAL = MODE == kDual;
    extern __shared__ __align__(16) uint8_t table_smem[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t tab0 = uint32_t(__cvta_generic_to_shared(table_smem));
    // Most bit patterns need no evaluation, because silu_f32 / gelu_f32 return a value known in advance there
    // (a warp's 32 consecutive patterns share sign and exponent, so the branch is uniform):
    //   2^-124 <= |h| < 2^-26: both give h / 2 after the rounding to bf16 (the sigmoid / Phi factor is 1/2 to
    //                          far below a bf16 half-step);
    //   h >= 32 (SiLU), h >= 16 (GELU): h itself (exp(-h), erfc(h / sqrt 2) are below fp32's resolution of 1);
    //   h <= -128 (SiLU), h <= -16 (GELU): -0 (the exponential has underflowed to zero).
    // NaN and infinities go through the functions.  The test that compares this variant with the arithmetic one
    // on all 65536 patterns holds these statements to the bit.
    const bool is_silu = prm.act == 1;
    for (uint32_t b = threadIdx.x; b < 65536u; b += kTableThreads) {
        const uint32_t e = (b >> 7) & 0xFFu, neg = b >> 15;
        uint32_t out;
        if (e >= 3u && e <= 100u) {
            out = b - 0x80u;                                  // exponent - 1
        } else if (e != 255u && !neg && e >= (is_silu ? 132u : 131u)) {
            out = b;
        } else if (e != 255u && neg && e >= (is_silu ? 134u : 131u)) {
            out = 0x8000u;
        } else {
            const float h = __uint_as_float(b << 16);
            const float a = is_silu ? silu_f32(h) : gelu_f32(h);
            const __nv_bfloat16 r = __float2bfloat16_rn(a);
            out = *reinterpret_cast<const unsigned short *>(&r);
        }
        reinterpret_cast<unsigned short *>(table_smem)[b] = static_cast<unsigned short>(out);
    }
    // the table depends on nothing in memory: it is built before the wait for the previous kernel of the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();
    auto lookup = [&](uint32_t bits16) -> float {       // bits of a bf16 pre-activation -> stored activation as fp32
        uint32_t v;
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(tab0 + (bits16 << 1)));
        return __uint_as_float(v << 16);
    };

    const SegBounds &sb = prm.sb;
    const int64_t M = prm.M;
    const int R = prm.R;
    const uint32_t g = blockIdx.x * kTableThreads + threadIdx.x;
    const uint32_t r0 = g / uint32_t(prm.V);
    if (r0 >= uint32_t(R) || int64_t(r0) >= M) return;
    const int k0 = int(g - r0 * uint32_t(prm.V)) * kVec;     // the host checked: every chunk lies in one K-segment
    int p = 0;
    while (p + 1 < sb.P && k0 >= sb.kb[p + 1]) p++;

    using Tin = __nv_bfloat16;
    const Tin *src = static_cast<const Tin *>(prm.X) + int64_t(r0) * prm.ld + k0;
    uint8_t *dp = prm.c_pos + int64_t(r0) * prm.ldc + k0;
    uint8_t *dn = DUAL ? prm.c_neg + int64_t(r0) * prm.ldc + k0 : nullptr;
    const int64_t src_step = int64_t(R) * prm.ld, dst_step = int64_t(R) * prm.ldc;
    float mreg[kVec];
#pragma unroll
    for (int i = 0; i < kVec; i++) mreg[i] = prm.mult ? __ldg(prm.mult + k0 + i) : 1.0f;
    const SegConst cp = seg_const(__ldg(prm.s_pos + p));
    const SegConst cn = seg_const(DUAL ? __ldg(prm.s_neg + p) : 1.0f);
    const bool fast = cp.fast && cn.fast && !(DUAL && CODE == SQ_CODE_INT8 && prm.lo != -128);

    const uint32_t ring0 = tab0 + uint32_t(kTableBytes) + threadIdx.x * 16u;
    auto slot_addr = [&](int slot, int v) { return ring0 + uint32_t((slot * 2 + v) * kTableThreads) * 16u; };
    auto copy_row = [&](const Tin *row_src, int slot, bool valid) {          // one commit group per call, always
        if (valid) {
#pragma unroll
            for (int v = 0; v < 2; v++)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(slot_addr(slot, v)),
                             "l"(reinterpret_cast<const char *>(row_src) + 16 * v) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
#pragma unroll
    for (int d = 0; d < kTableDepth - 1; d++) copy_row(src + int64_t(d) * src_step, d, int64_t(r0) + int64_t(d) * R < M);
    int slot = 0;
    for (int64_t row = r0; row < M; row += R) {
        const int ahead = slot == 0 ? kTableDepth - 1 : slot - 1;
        copy_row(src + int64_t(kTableDepth - 1) * src_step, ahead, row + int64_t(kTableDepth - 1) * R < M);
        asm volatile("cp.async.wait_group %0;" ::"n"(kTableDepth - 1) : "memory");
        uint32_t w[8];
#pragma unroll
        for (int v = 0; v < 2; v++)
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w[4 * v]), "=r"(w[4 * v + 1]), "=r"(w[4 * v + 2]), "=r"(w[4 * v + 3])
                         : "r"(slot_addr(slot, v)) : "memory");
        slot = slot + 1 == kTableDepth ? 0 : slot + 1;
        uint32_t wp[4], wn[4];
#pragma unroll
        for (int g4 = 0; g4 < 4; g4++) {
            float x[4];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const uint32_t word = w[2 * g4 + (i >> 1)];
                x[i] = __fmul_rn(lookup((i & 1) ? (word >> 16) : (word & 0xFFFFu)), mreg[4 * g4 + i]);
            }
            if (fast) {
                quant4<CODE, MODE>(x, cp, cn, float(prm.hi), 0, wp[g4], wn[g4]);
            } else {
                wp[g4] = wn[g4] = 0u;
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    uint32_t a, b;
                    quant1<CODE, MODE>(x[i], cp.s, cn.s, 0, prm.lo, prm.hi, a, b);
                    wp[g4] |= (a & 0xFFu) << (8 * i);
                    wn[g4] |= (b & 0xFFu) << (8 * i);
                }
            }
        }
        *reinterpret_cast<uint4 *>(dp) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
        if (DUAL) *reinterpret_cast<uint4 *>(dn) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
        src += src_step;
        dp += dst_step;
        if (DUAL) dn += dst_step;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ----------------------------------------------------------------------------- per-row scales (W4A8)
// App. B "Extra Hyperparameter Settings": 4-bit weights are quantized per channel, activations dynamically per
// token.  One CTA per row: the row is read once into registers (up to kRowChunks 16-element chunks per thread),
// its extrema per K-segment are reduced in shared memory, the scales (one IEEE division each) are written out,
// and the codes are made from the registers with the same quantizer as everywhere else.
constexpr int kRowChunks = 4;                       // K <= 256 threads x 4 chunks x 16 = 16384

__device__ __forceinline__ uint32_t ord_enc(float f)     // monotone map float -> uint32
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord_dec(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

// largest and smallest of the 16 elements of a chunk (bf16: on packed pairs, two elements per instruction)
__device__ __forceinline__ void chunk_extrema(const Raw16<float> &r, float &mx, float &mn)
{
    mx = -INFINITY; mn = INFINITY;
#pragma unroll
    for (int v = 0; v < 4; v++) {
        mx = fmaxf(fmaxf(mx, r.v[v].x), fmaxf(r.v[v].y, fmaxf(r.v[v].z, r.v[v].w)));
        mn = fminf(fminf(mn, r.v[v].x), fminf(r.v[v].y, fminf(r.v[v].z, r.v[v].w)));
    }
}
__device__ __forceinline__ void chunk_extrema(const Raw16<__nv_bfloat16> &r, float &mx, float &mn)
{
    const uint32_t w[8] = {r.v[0].x, r.v[0].y, r.v[0].z, r.v[0].w, r.v[1].x, r.v[1].y, r.v[1].z, r.v[1].w};
    __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162 *>(&w[0]), lo = hi;
#pragma unroll
    for (int i = 1; i < 8; i++) {
        const __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162 *>(&w[i]);
        hi = __hmax2(hi, x);
        lo = __hmin2(lo, x);
    }
    mx = fmaxf(__low2float(hi), __high2float(hi));
    mn = fminf(__low2float(lo), __high2float(lo));
}

template <typename Tin, bool DUAL>
__global__ void __launch_bounds__(kThreads)
quantize_per_row_kernel(const Tin *__restrict__ X, int K, int64_t ld, const SegBounds sb, float q_max, float q_min_abs,
                        float *__restrict__ s_pos, float *__restrict__ s_neg, uint8_t *__restrict__ c_pos,
                        uint8_t *__restrict__ c_neg, int64_t ldc)
{
    __shared__ uint32_t sh_max[SQ_MAX_P], sh_min[SQ_MAX_P];
    __shared__ float sh_sp[SQ_MAX_P], sh_sn[SQ_MAX_P];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t row = blockIdx.x;
    const int P = sb.P;
    // One K-segment (the usual case) needs ONE block barrier: every warp leaves its extrema in a slot, and after the
    // barrier every thread reduces the slots and computes the scales itself.  Several K-segments go through
    // shared-memory words per segment (three barriers).
    const bool one = P == 1;
    __shared__ float sh_wmax[kThreads / 32], sh_wmin[kThreads / 32];
    float one_sp = 1.0f, one_sn = 1.0f, tail_mx = -INFINITY, tail_mn = INFINITY;
    if (!one) {
        for (int i = threadIdx.x; i < P; i += blockDim.x) { sh_max[i] = 0u; sh_min[i] = 0xFFFFFFFFu; }
        __syncthreads();
    }
    const Tin *src = X + row * ld;
    Raw16<Tin> raw[kRowChunks];
    int seg[kRowChunks];                            // K-segment of a whole chunk, -1: straddles a bound or the row end
#pragma unroll
    for (int c = 0; c < kRowChunks; c++) {
        const int k0 = (int(threadIdx.x) + c * int(blockDim.x)) * kVec;
        seg[c] = -2;                                // beyond the row
        if (k0 >= K) continue;
        int p = 0;
        while (p + 1 < P && k0 >= sb.kb[p + 1]) p++;
        if (k0 + kVec <= sb.kb[p + 1]) {
            seg[c] = p;
            load16(src + k0, raw[c]);
        } else {
            seg[c] = -1;
            const int n = min(kVec, K - k0);
            for (int i = 0; i < n; i++) {
                while (p + 1 < P && k0 + i >= sb.kb[p + 1]) p++;
                const float x = load1(src + k0 + i);
                if (one) {
                    tail_mx = fmaxf(tail_mx, x);
                    tail_mn = fminf(tail_mn, x);
                } else {
                    atomicMax(&sh_max[p], ord_enc(x));
                    atomicMin(&sh_min[p], ord_enc(x));
                }
            }
        }
    }
    if (one) {
        float mx = tail_mx, mn = tail_mn;
#pragma unroll
        for (int c = 0; c < kRowChunks; c++) {
            if (seg[c] >= 0) {
                float cx, cm;
                chunk_extrema(raw[c], cx, cm);
                mx = fmaxf(mx, cx);
                mn = fminf(mn, cm);
            }
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
        }
        if ((threadIdx.x & 31) == 0) { sh_wmax[threadIdx.x >> 5] = mx; sh_wmin[threadIdx.x >> 5] = mn; }
        __syncthreads();
        mx = sh_wmax[0]; mn = sh_wmin[0];
        for (int w = 1; w < int(blockDim.x >> 5); w++) { mx = fmaxf(mx, sh_wmax[w]); mn = fminf(mn, sh_wmin[w]); }
        if (DUAL) {
            const float h = fmaxf(mx, 0.0f), l = fmaxf(-mn, 0.0f);
            one_sp = h > 0.0f ? __fdiv_rn(h, q_max) : 1.0f;
            one_sn = l > 0.0f ? __fdiv_rn(l, q_min_abs) : 1.0f;
            if (threadIdx.x == 0) s_neg[row] = one_sn;
        } else {
            const float a = fmaxf(fabsf(mx), fabsf(mn));
            one_sp = a > 0.0f ? __fdiv_rn(a, q_max) : 1.0f;
        }
        if (threadIdx.x == 0) s_pos[row] = one_sp;
    } else {
    // Extrema: where the 32 chunks of a warp lie in one K-segment (512 consecutive columns: the usual case) they are
    // reduced with shuffles and one lane updates the shared words; same-address shared atomics from every thread
    // serialise, and were most of this kernel's time.  Every lane takes part in the votes and shuffles.
#pragma unroll
    for (int c = 0; c < kRowChunks; c++) {
        float mx = -INFINITY, mn = INFINITY;
        if (seg[c] >= 0) chunk_extrema(raw[c], mx, mn);
        const int s0 = __shfl_sync(0xFFFFFFFFu, seg[c], 0);
        const bool uniform = __all_sync(0xFFFFFFFFu, seg[c] == s0) && s0 >= 0;
        if (uniform) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
                mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
            }
            if ((threadIdx.x & 31) == 0) {
                atomicMax(&sh_max[s0], ord_enc(mx));
                atomicMin(&sh_min[s0], ord_enc(mn));
            }
        } else if (seg[c] >= 0) {
            atomicMax(&sh_max[seg[c]], ord_enc(mx));
            atomicMin(&sh_min[seg[c]], ord_enc(mn));
        }
    }
    __syncthreads();
    for (int p = threadIdx.x; p < P; p += blockDim.x) {
        const float mx = ord_dec(sh_max[p]), mn = ord_dec(sh_min[p]);
        float sp, sn = 1.0f;
        if (DUAL) {
            const float hi = fmaxf(mx, 0.0f), lo = fmaxf(-mn, 0.0f);
            sp = hi > 0.0f ? __fdiv_rn(hi, q_max) : 1.0f;
            sn = lo > 0.0f ? __fdiv_rn(lo, q_min_abs) : 1.0f;
            s_neg[row * P + p] = sn;
        } else {
            const float a = fmaxf(fabsf(mx), fabsf(mn));
            sp = a > 0.0f ? __fdiv_rn(a, q_max) : 1.0f;
        }
        s_pos[row * P + p] = sp;
        sh_sp[p] = sp;
        sh_sn[p] = sn;
    }
    __syncthreads();
    }
    const int hi = int(q_max), lo = DUAL ? -int(q_min_abs) : -int(q_max);
    constexpr int MODE = DUAL ? kDual : kSingle;
    SegConst cp, cn;
    int const_seg = -1;
#pragma unroll
    for (int c = 0; c < kRowChunks; c++) {
        const int k0 = (int(threadIdx.x) + c * int(blockDim.x)) * kVec;
        if (seg[c] == -2) continue;
        uint8_t *dp = c_pos + row * ldc + k0;
        uint8_t *dn = DUAL ? c_neg + row * ldc + k0 : nullptr;
        bool done = false;
        if (seg[c] >= 0) {
            if (seg[c] != const_seg) {              // constants are remade only when the chunk's K-segment changes
                cp = seg_const(one ? one_sp : sh_sp[seg[c]]);
                cn = seg_const(DUAL ? (one ? one_sn : sh_sn[seg[c]]) : 1.0f);
                const_seg = seg[c];
            }
            if (cp.fast && cn.fast && !(DUAL && lo != -128)) {
                uint32_t wp[4], wn[4];
#pragma unroll
                for (int g4 = 0; g4 < 4; g4++) {
                    float x[4];
                    get4(raw[c], g4, x);
                    quant4<SQ_CODE_INT8, MODE>(x, cp, cn, float(hi), 0, wp[g4], wn[g4]);
                }
                *reinterpret_cast<uint4 *>(dp) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
                if (DUAL) *reinterpret_cast<uint4 *>(dn) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
                done = true;
            }
        }
        if (!done) {
            const int n = min(kVec, K - k0);
            int p = 0;
            for (int i = 0; i < n; i++) {
                while (p + 1 < P && k0 + i >= sb.kb[p + 1]) p++;
                uint32_t a, b;
                quant1<SQ_CODE_INT8, MODE>(load1(src + k0 + i), one ? one_sp : sh_sp[p], one ? one_sn : sh_sn[p], 0, lo, hi, a, b);
                dp[i] = uint8_t(a);
                if (DUAL) dn[i] = uint8_t(b);
            }
        }
    }
}

// int8 codes in [-8, 7] <-> two 4-bit codes per byte (code 2j in the low nibble); 16 codes per thread
__global__ void __launch_bounds__(kThreads)
pack_w4_kernel(uint8_t *__restrict__ w8, int64_t ld8, int64_t N, int K, uint8_t *__restrict__ w4, int64_t ld4, int unpack)
{
    const int V = K / kVec;
    const int64_t idx = int64_t(blockIdx.x) * kThreads + threadIdx.x;
    if (idx >= N * V) return;
    const int64_t n = idx / V;
    const int k0 = int(idx - n * V) * kVec;
    if (!unpack) {
        const uint4 v = *reinterpret_cast<const uint4 *>(w8 + n * ld8 + k0);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[2];
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const uint32_t a = w[2 * h], b = w[2 * h + 1];          // 4 codes each
            const uint32_t pa = (a & 0xF) | ((a >> 4) & 0xF0) | ((a >> 8) & 0xF00) | ((a >> 12) & 0xF000);
            const uint32_t pb = (b & 0xF) | ((b >> 4) & 0xF0) | ((b >> 8) & 0xF00) | ((b >> 12) & 0xF000);
            o[h] = pa | (pb << 16);
        }
        *reinterpret_cast<uint2 *>(w4 + n * ld4 + k0 / 2) = make_uint2(o[0], o[1]);
    } else {
        const uint2 v = *reinterpret_cast<const uint2 *>(w4 + n * ld4 + k0 / 2);
        const uint32_t in[2] = {v.x, v.y};
        uint32_t o[4];
#pragma unroll
        for (int h = 0; h < 2; h++) {
#pragma unroll
            for (int t = 0; t < 2; t++) {
                const uint32_t hw = (in[h] >> (16 * t)) & 0xFFFFu;   // 4 nibbles
                uint32_t bytes = (hw & 0xF) | ((hw & 0xF0) << 4) | ((hw & 0xF00) << 8) | ((hw & 0xF000) << 12);
                bytes |= (bytes & 0x08080808u) * 0x1Eu;              // sign-extend each nibble: bit 3 copied into bits 4..7
                o[2 * h + t] = bytes;
            }
        }
        *reinterpret_cast<uint4 *>(w8 + n * ld8 + k0) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

template <typename Tin, int CODE, int MODE>
sq_status prepare_t(QuantLaunch &L)
{
    // V chunks per row; R rows in flight: enough threads to fill every SM several times over, and a row count per
    // thread that the rows divide into evenly
    QuantParams &prm = L.prm;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return SQ_ERR_CUDA;
    const bool pre = prm.act != 0 || prm.mult != nullptr;
    const int64_t V = (prm.K + kVec - 1) / kVec;
    const int64_t target_threads = int64_t(sms) * kThreads * (pre ? 3 : kBlocksPerSm);
    int64_t iters = (prm.M * V + target_threads - 1) / target_threads;
    if (iters < 1) iters = 1;
    const int64_t R = (prm.M + iters - 1) / iters;
    const int64_t blocks = (R * V + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF || R * V > 0xFFFFFFFFll || V > 0x7FFFFFFF || R > 0x7FFFFFFF) return SQ_ERR_SHAPE;
    prm.V = int(V);
    prm.R = int(R);
    L.blocks = unsigned(blocks);
    // fp32 input: 64-byte chunks, so half the depth for the same shared memory
    const bool deep = iters >= 10 && sizeof(Tin) == 2;
    if (prm.act == SQ_ACT_GEGLU)
        L.kernel = deep ? reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 2, 4>)
                        : reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 2, 2>);
    else if (pre)
        L.kernel = deep ? reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 1, 4>)
                        : reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 1, 2>);
    else
        L.kernel = deep ? reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 0, 4>)
                        : reinterpret_cast<const void *>(quantize_kernel<Tin, CODE, MODE, 0, 2>);
    return SQ_OK;
}

template <typename Tin>
sq_status prepare_mode(QuantLaunch &L, sq_code code, int mode)
{
    if (mode == kZeroPoint) return prepare_t<Tin, SQ_CODE_INT8, kZeroPoint>(L);
    if (code == SQ_CODE_INT8)
        return mode == kDual ? prepare_t<Tin, SQ_CODE_INT8, kDual>(L) : prepare_t<Tin, SQ_CODE_INT8, kSingle>(L);
    return mode == kDual ? prepare_t<Tin, SQ_CODE_E4M3, kDual>(L) : prepare_t<Tin, SQ_CODE_E4M3, kSingle>(L);
}

// The table variant of the fused activation: bf16 input, SiLU or GELU, every 16-element chunk inside one K-segment,
// and enough elements for the table's set-up time not to count.  Returns false where it does not apply.
std::atomic<int> g_table_mode{0};        // test hook: 0 automatic, 1 always where possible, 2 never
constexpr int64_t kTableMinSilu = int64_t(16) << 20, kTableMinGelu = int64_t(8) << 20;   // measured break-even points
bool prepare_table(QuantLaunch &L, sq_dtype dt, sq_code code, int mode)
{
    QuantParams &prm = L.prm;
    const int tm = g_table_mode.load(std::memory_order_relaxed);
    if (tm == 2 || dt != SQ_BF16 || mode == kZeroPoint || prm.row_segments) return false;
    if (prm.act != SQ_ACT_SILU && prm.act != SQ_ACT_GELU) return false;
    if (prm.K % kVec != 0) return false;
    for (int p = 1; p < prm.sb.P; p++)
        if (prm.sb.kb[p] % kVec != 0) return false;
    if (tm != 1 && prm.M * int64_t(prm.K) < (prm.act == SQ_ACT_SILU ? kTableMinSilu : kTableMinGelu)) return false;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return false;
    const int64_t V = prm.K / kVec;
    const int64_t threads = int64_t(sms) * kTableThreads;                 // one CTA per SM
    int64_t iters = (prm.M * V + threads - 1) / threads;
    if (iters < 1) iters = 1;
    const int64_t R = (prm.M + iters - 1) / iters;
    const int64_t blocks = (R * V + kTableThreads - 1) / kTableThreads;
    if (blocks > 0x7FFFFFFF || R * V > 0xFFFFFFFFll || V > 0x7FFFFFFF || R > 0x7FFFFFFF) return false;
    const void *kern = nullptr;
    if (code == SQ_CODE_INT8)
        kern = mode == kDual ? reinterpret_cast<const void *>(quantize_table_kernel<SQ_CODE_INT8, kDual>)
                             : reinterpret_cast<const void *>(quantize_table_kernel<SQ_CODE_INT8, kSingle>);
    else
        kern = mode == kDual ? reinterpret_cast<const void *>(quantize_table_kernel<SQ_CODE_E4M3, kDual>)
                             : reinterpret_cast<const void *>(quantize_table_kernel<SQ_CODE_E4M3, kSingle>);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kTableSmem)) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    prm.V = int(V);
    prm.R = int(R);
    L.blocks = unsigned(blocks);
    L.kernel = kern;
    L.threads = kTableThreads;
    L.smem = unsigned(kTableSmem);
    return true;
}

}  // namespace

void set_quantize_table_mode(int mode) { g_table_mode.store(mode, std::memory_order_relaxed); }

sq_status prepare_quantize(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                           const float *s_pos, const float *s_neg, const int32_t *zero_point, int row_segments,
                           sq_code code, float q_max, float q_min_abs, int act, const float *mult,
                           void *c_pos, void *c_neg, int64_t ldc, QuantLaunch *out)
{
    QuantParams &prm = out->prm;
    prm = QuantParams{};
    out->threads = 0;
    out->smem = 0;
    prm.X = X; prm.M = M; prm.K = int(K); prm.ld = ld;
    prm.sb = sb;
    prm.s_pos = s_pos; prm.s_neg = s_neg; prm.zp = zero_point;
    prm.row_segments = row_segments;
    // dual: codes in [-|q_min|, q_max]; single scale: symmetric [-q_max, q_max]; zero-point: the whole int8 range
    prm.hi = int(q_max);
    prm.lo = (s_neg || zero_point) ? -int(q_min_abs) : -int(q_max);
    prm.c_pos = static_cast<uint8_t *>(c_pos); prm.c_neg = static_cast<uint8_t *>(c_neg); prm.ldc = ldc;
    prm.act = act; prm.mult = mult;
    const int mode = zero_point ? kZeroPoint : (s_neg ? kDual : kSingle);
    if (prepare_table(*out, dt, code, mode)) return SQ_OK;
    return dt == SQ_F32 ? prepare_mode<float>(*out, code, mode) : prepare_mode<__nv_bfloat16>(*out, code, mode);
}

sq_status run_quantize(const QuantLaunch &L, cudaStream_t st)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(L.blocks);
    cfg.blockDim = dim3(L.threads ? L.threads : unsigned(kThreads));
    cfg.dynamicSmemBytes = L.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void *args[1] = {const_cast<QuantParams *>(&L.prm)};
    const cudaError_t e = cudaLaunchKernelExC(&cfg, L.kernel, args);
    count_launch();
    if (e != cudaSuccess) { note_cuda_error(e); return SQ_ERR_CUDA; }
    return SQ_OK;
}

sq_status launch_quantize(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                          const float *s_pos, const float *s_neg, const int32_t *zero_point, int row_segments,
                          sq_code code, float q_max, float q_min_abs, int act, const float *mult,
                          void *c_pos, void *c_neg, int64_t ldc, cudaStream_t st)
{
    QuantLaunch L;
    const sq_status s = prepare_quantize(X, dt, M, K, ld, sb, s_pos, s_neg, zero_point, row_segments, code, q_max,
                                         q_min_abs, act, mult, c_pos, c_neg, ldc, &L);
    return s == SQ_OK ? run_quantize(L, st) : s;
}

sq_status launch_quantize_per_row(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                                  int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                                  void *c_pos, void *c_neg, int64_t ldc, cudaStream_t st)
{
    const int64_t V = (K + kVec - 1) / kVec;
    if (V > int64_t(kThreads) * kRowChunks) return SQ_ERR_UNSUPPORTED;      // the row is held in registers
    if (M > 0x7FFFFFFF) return SQ_ERR_SHAPE;
    int threads = int((V + kRowChunks - 1) / kRowChunks);
    threads = (threads + 31) / 32 * 32;
    if (threads < 32) threads = 32;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(M));
    cfg.blockDim = dim3(unsigned(threads));
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    uint8_t *cp = static_cast<uint8_t *>(c_pos), *cn = static_cast<uint8_t *>(c_neg);
    const int Ki = int(K);
    cudaError_t e;
    if (dt == SQ_F32) {
        const float *x = static_cast<const float *>(X);
        e = dual ? cudaLaunchKernelEx(&cfg, quantize_per_row_kernel<float, true>, x, Ki, ld, sb, q_max, q_min_abs, s_pos, s_neg, cp, cn, ldc)
                 : cudaLaunchKernelEx(&cfg, quantize_per_row_kernel<float, false>, x, Ki, ld, sb, q_max, q_min_abs, s_pos, s_neg, cp, cn, ldc);
    } else {
        const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(X);
        e = dual ? cudaLaunchKernelEx(&cfg, quantize_per_row_kernel<__nv_bfloat16, true>, x, Ki, ld, sb, q_max, q_min_abs, s_pos, s_neg, cp, cn, ldc)
                 : cudaLaunchKernelEx(&cfg, quantize_per_row_kernel<__nv_bfloat16, false>, x, Ki, ld, sb, q_max, q_min_abs, s_pos, s_neg, cp, cn, ldc);
    }
    count_launch();
    if (e != cudaSuccess) { note_cuda_error(e); return SQ_ERR_CUDA; }
    return SQ_OK;
}

sq_status launch_pack_w4(const void *Wq8, int64_t ld8, int64_t N, int64_t K, void *Wq4, int64_t ld4, int unpack,
                         cudaStream_t st)
{
    const int64_t blocks = (N * (K / kVec) + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return SQ_ERR_SHAPE;
    pack_w4_kernel<<<unsigned(blocks), kThreads, 0, st>>>(static_cast<uint8_t *>(const_cast<void *>(Wq8)), ld8, N, int(K),
                                                          static_cast<uint8_t *>(Wq4), ld4, unpack);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error(e); return SQ_ERR_CUDA; }
    return SQ_OK;
}

}  // namespace sq
