// Activation / weight quantization kernels (Sec. 3 uniform quantizer, Sec. 4.3.2 Q_dual and polarity
// split, Sec. 4.2.2 one scale per segment).  HBM-streaming: every thread converts 16 consecutive
// elements of one row (128-bit loads, one 128-bit store per code matrix).  The codes are those of
// "one IEEE fp32 division, round half to even, clip"; the common case computes them with a handful of
// full-rate fp32 instructions per element (see SegConst) so that the pass stays memory bound.
#include <cuda_bf16.h>
#include "sq_common.cuh"

namespace sq {
namespace {

constexpr int kThreads = 256;
constexpr int kVec = 16;   // elements per thread

__device__ __forceinline__ void load16(const float *p, float (&x)[kVec])
{
    const float4 *q = reinterpret_cast<const float4 *>(p);
#pragma unroll
    for (int i = 0; i < 4; i++) {
        float4 v = __ldg(q + i);
        x[4 * i + 0] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
    }
}

__device__ __forceinline__ void load16(const __nv_bfloat16 *p, float (&x)[kVec])
{
    const uint4 *q = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int i = 0; i < 2; i++) {
        uint4 v = __ldg(q + i);
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; j++) {
            x[8 * i + 2 * j + 0] = __uint_as_float(w[j] << 16);
            x[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
    }
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

// One element -> (code for the positive / only matrix, code for the negative matrix), as bytes.
// Reference form: one IEEE division, round half to even, clip.  Used where a vector straddles a
// segment bound or the end of a row, and for scales outside the range of the fast form below.
template <int CODE, bool DUAL>
__device__ __forceinline__ void quant1(float x, float sp, float sn, int lo, int hi, uint32_t &cp, uint32_t &cn)
{
    if (CODE == SQ_CODE_INT8) {
        float s = DUAL ? (x >= 0.0f ? sp : sn) : sp;
        int c = __float2int_rn(__fdiv_rn(x, s));      // IEEE divide, round half to even, saturating convert
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

// Per-segment constants of the fast form.  The quotient x / s is obtained, correctly rounded, from the
// correctly rounded reciprocal r = RN(1/s) by one multiply and two FMAs:
//   q0 = RN(x r),  e = x - q0 s (exact in one FMA),  q = RN(q0 + e r)
// which equals RN(x / s) when nothing over- or underflows on the way.  To rule that out, and to get the
// polarity split for free, the input is first mapped to u = sat(x / L) in [0, 1] by one saturating FMA,
// L = 2^(exponent(s) + 11) >= 1024 s.  L is a power of two, so x / L is exact and u / (s / L) has the
// bits of x / s; negative x give u = 0 (the other polarity's zero code) and x > L, which is clipped to
// the end of the code range anyway, gives u = 1.  A quotient too small to be normal rounds to code 0
// whatever its last bits are.  The fast form is taken for 2^-100 <= s <= 2^100.
struct SegConst {
    float inv_l;       // 1 / L
    float s_l, r_l;    // s / L and RN(L / s) = RN(1 / s) L
    int fast;
};
__device__ __forceinline__ SegConst seg_const(float s)
{
    SegConst c;
    c.fast = (s >= 7.8886090522101181e-31f && s <= 1.2676506002282294e+30f) ? 1 : 0;
    const uint32_t l_bits = (__float_as_uint(s) & 0x7F800000u) + (11u << 23);
    const float l = __uint_as_float(l_bits);
    c.inv_l = __uint_as_float((254u << 23) - l_bits);
    c.s_l = s * c.inv_l;
    c.r_l = __frcp_rn(s) * l;
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
// two correctly rounded quotients x / s from r = RN(1/s): q0 = RN(x r), e = x - q0 s, q = RN(q0 + e r)
__device__ __forceinline__ uint64_t div2_rn_fast(uint64_t x2, uint64_t neg_s2, uint64_t r2)
{
    const uint64_t q0 = mul2(x2, r2);
    const uint64_t e = fma2(q0, neg_s2, x2);
    return fma2(e, r2, q0);
}

constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23: v + magic rounds v to an integer, half to even

// 16 elements of one K-segment -> packed codes.  int8: clip in fp32 (the bounds are integers, so
// clip-then-round equals round-then-clip), add the magic constant, and the low byte of the sum's bit
// pattern is the two's-complement code.  Dual: the positive matrix quantizes max(x, 0) = L sat(x / L),
// the negative one min(x, 0) = -L sat(-x / L), each with its own constants, which reproduces the
// per-element polarity select.  Single scale: |x| is quantized and the sign put back when rounding.
template <int CODE, bool DUAL>
__device__ __forceinline__ void quant16(const float (&x)[kVec], const SegConst &cp, const SegConst &cn, float lo,
                                        float hi, uint32_t (&wp)[4], uint32_t (&wn)[4])
{
    uint32_t bp[kVec], bn[kVec];
    const uint64_t rp2 = pack2(cp.r_l, cp.r_l), nsp2 = pack2(-cp.s_l, -cp.s_l);
    const uint64_t rn2 = pack2(-cn.r_l, -cn.r_l), nsn2 = pack2(cn.s_l, cn.s_l);   // negated: quotients <= 0
    const uint64_t magic2 = pack2(kRoundMagic, kRoundMagic);
#pragma unroll
    for (int i = 0; i < kVec; i += 2) {
        float a0, a1;
        if (DUAL) {
            const uint64_t qp2 = div2_rn_fast(pack2(fma_sat(x[i], cp.inv_l, 0.0f), fma_sat(x[i + 1], cp.inv_l, 0.0f)), nsp2, rp2);
            const uint64_t qn2 = div2_rn_fast(pack2(fma_sat(x[i], -cn.inv_l, 0.0f), fma_sat(x[i + 1], -cn.inv_l, 0.0f)), nsn2, rn2);
            if (CODE == SQ_CODE_INT8) {
                unpack2(qp2, a0, a1);
                unpack2(add2(pack2(fminf(a0, hi), fminf(a1, hi)), magic2), a0, a1);
                bp[i] = __float_as_uint(a0); bp[i + 1] = __float_as_uint(a1);
                unpack2(qn2, a0, a1);
                unpack2(add2(pack2(fmaxf(a0, lo), fmaxf(a1, lo)), magic2), a0, a1);
                bn[i] = __float_as_uint(a0); bn[i + 1] = __float_as_uint(a1);
            } else {
                unpack2(qp2, a0, a1);
                bp[i] = __float_as_uint(a0); bp[i + 1] = __float_as_uint(a1);
                unpack2(qn2, a0, a1);
                bn[i] = __float_as_uint(a0); bn[i + 1] = __float_as_uint(a1);
            }
        } else {
            const uint64_t q2 = div2_rn_fast(pack2(fma_sat(fabsf(x[i]), cp.inv_l, 0.0f), fma_sat(fabsf(x[i + 1]), cp.inv_l, 0.0f)), nsp2, rp2);
            unpack2(q2, a0, a1);
            if (CODE == SQ_CODE_INT8) {                  // the range is symmetric: clip |q|, round with the sign of x
                a0 = fmaf(fminf(a0, hi), copysignf(1.0f, x[i]), kRoundMagic);
                a1 = fmaf(fminf(a1, hi), copysignf(1.0f, x[i + 1]), kRoundMagic);
            } else {
                a0 = copysignf(a0, x[i]);
                a1 = copysignf(a1, x[i + 1]);
            }
            bp[i] = __float_as_uint(a0); bp[i + 1] = __float_as_uint(a1);
        }
    }
#pragma unroll
    for (int g = 0; g < 4; g++) {
        if (CODE == SQ_CODE_INT8) {
            wp[g] = __byte_perm(__byte_perm(bp[4 * g], bp[4 * g + 1], 0x0040), __byte_perm(bp[4 * g + 2], bp[4 * g + 3], 0x0040), 0x5410);
            if (DUAL)
                wn[g] = __byte_perm(__byte_perm(bn[4 * g], bn[4 * g + 1], 0x0040), __byte_perm(bn[4 * g + 2], bn[4 * g + 3], 0x0040), 0x5410);
        } else {
            uint32_t w = cvt_e4m3x2(__uint_as_float(bp[4 * g]), __uint_as_float(bp[4 * g + 1])) |
                         (cvt_e4m3x2(__uint_as_float(bp[4 * g + 2]), __uint_as_float(bp[4 * g + 3])) << 16);
            wp[g] = w & ~(__vcmpeq4(w & 0x7F7F7F7Fu, 0u) & 0x80808080u);      // -0 is stored as +0
            if (DUAL) {
                w = cvt_e4m3x2(__uint_as_float(bn[4 * g]), __uint_as_float(bn[4 * g + 1])) |
                    (cvt_e4m3x2(__uint_as_float(bn[4 * g + 2]), __uint_as_float(bn[4 * g + 3])) << 16);
                wn[g] = w & ~(__vcmpeq4(w & 0x7F7F7F7Fu, 0u) & 0x80808080u);
            }
        }
    }
}

template <typename Tin, int CODE, bool DUAL>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const Tin *__restrict__ X, int64_t M, int K, int64_t ld, const SegBounds sb,
                const float *__restrict__ s_pos, const float *__restrict__ s_neg, int row_segments,
                int lo, int hi, uint8_t *__restrict__ c_pos, uint8_t *__restrict__ c_neg, int64_t ldc)
{
    // Programmatic dependent launch: this kernel may be scheduled while the previous kernel of the stream
    // winds down, and lets the next one be scheduled while its own last blocks run; nothing in global
    // memory is touched before the previous kernel has completed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int V = (K + kVec - 1) / kVec;
    const int64_t idx = int64_t(blockIdx.x) * kThreads + threadIdx.x;
    if (idx >= M * int64_t(V)) return;
    const int64_t row = idx / V;
    const int k0 = int(idx - row * V) * kVec;

    // segment of this vector (bounds come with the kernel parameters); the scale loads below do not
    // depend on the data loads, so both are in flight together
    const int Qs = row_segments ? sb.Q : 1;
    int q = 0;
    if (row_segments) while (q + 1 < sb.Q && row >= sb.nb[q + 1]) q++;
    int p = 0;
    while (p + 1 < sb.P && k0 >= sb.kb[p + 1]) p++;
    const bool whole = k0 + kVec <= sb.kb[p + 1];            // vector inside one K-segment (and inside K)

    const Tin *src = X + row * ld + k0;
    uint8_t *dp = c_pos + row * ldc + k0;
    uint8_t *dn = DUAL ? c_neg + row * ldc + k0 : nullptr;

    float x[kVec];
    if (whole) load16(src, x);
    const SegConst cp = seg_const(__ldg(s_pos + p * Qs + q));
    const SegConst cn = seg_const(DUAL ? __ldg(s_neg + p * Qs + q) : 1.0f);
    if (whole && cp.fast && cn.fast) {
        uint32_t wp[4], wn[4];
        quant16<CODE, DUAL>(x, cp, cn, float(lo), float(hi), wp, wn);
        *reinterpret_cast<uint4 *>(dp) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
        if (DUAL) *reinterpret_cast<uint4 *>(dn) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
    } else {                                    // segment bound or end of row inside the vector, or an extreme scale
        const int n = min(kVec, K - k0);
        for (int i = 0; i < n; i++) {
            while (p + 1 < sb.P && k0 + i >= sb.kb[p + 1]) p++;
            uint32_t a, b;
            quant1<CODE, DUAL>(load1(src + i), __ldg(s_pos + p * Qs + q), DUAL ? __ldg(s_neg + p * Qs + q) : 0.0f, lo, hi,
                               a, b);
            dp[i] = uint8_t(a);
            if (DUAL) dn[i] = uint8_t(b);
        }
    }
}

template <typename Tin, int CODE>
sq_status launch_t(const Tin *X, int64_t M, int64_t K, int64_t ld, const SegBounds &sb, const float *s_pos,
                   const float *s_neg, int row_segments, int lo, int hi, void *c_pos, void *c_neg,
                   int64_t ldc, cudaStream_t st)
{
    const int64_t V = (K + kVec - 1) / kVec;
    const int64_t blocks = (M * V + kThreads - 1) / kThreads;
    if (blocks > 0x7FFFFFFF) return SQ_ERR_SHAPE;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(blocks));
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int Ki = int(K);
    uint8_t *cp = static_cast<uint8_t *>(c_pos), *cn = static_cast<uint8_t *>(c_neg);
    const float *no_neg = nullptr;
    if (s_neg)
        cudaLaunchKernelEx(&cfg, quantize_kernel<Tin, CODE, true>, X, M, Ki, ld, sb, s_pos, s_neg, row_segments, lo, hi, cp, cn, ldc);
    else
        cudaLaunchKernelEx(&cfg, quantize_kernel<Tin, CODE, false>, X, M, Ki, ld, sb, s_pos, no_neg, row_segments, lo, hi, cp,
                           static_cast<uint8_t *>(nullptr), ldc);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

}  // namespace

sq_status launch_quantize(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                          const float *s_pos, const float *s_neg, int row_segments, sq_code code,
                          float q_max, float q_min_abs, void *c_pos, void *c_neg, int64_t ldc, cudaStream_t st)
{
    // dual: codes in [-|q_min|, q_max]; single scale: symmetric [-q_max, q_max]
    const int hi = int(q_max);
    const int lo = s_neg ? -int(q_min_abs) : -int(q_max);
    if (dt == SQ_F32) {
        const float *x = static_cast<const float *>(X);
        return code == SQ_CODE_INT8
                   ? launch_t<float, SQ_CODE_INT8>(x, M, K, ld, sb, s_pos, s_neg, row_segments, lo, hi, c_pos, c_neg, ldc, st)
                   : launch_t<float, SQ_CODE_E4M3>(x, M, K, ld, sb, s_pos, s_neg, row_segments, lo, hi, c_pos, c_neg, ldc, st);
    }
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(X);
    return code == SQ_CODE_INT8
               ? launch_t<__nv_bfloat16, SQ_CODE_INT8>(x, M, K, ld, sb, s_pos, s_neg, row_segments, lo, hi, c_pos, c_neg, ldc, st)
               : launch_t<__nv_bfloat16, SQ_CODE_E4M3>(x, M, K, ld, sb, s_pos, s_neg, row_segments, lo, hi, c_pos, c_neg, ldc, st);
}

}  // namespace sq
