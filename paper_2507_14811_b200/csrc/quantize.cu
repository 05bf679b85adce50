// Activation / weight quantization kernels (Sec. 3 uniform quantizer, Sec. 4.3.2 Q_dual and polarity
// split, Sec. 4.2.2 one scale per segment).  HBM-streaming: every thread converts 16 consecutive
// elements of one row (128-bit loads, one 128-bit store per code matrix).
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

template <typename Tin, int CODE, bool DUAL>
__global__ void __launch_bounds__(kThreads)
quantize_kernel(const Tin *__restrict__ X, int64_t M, int K, int64_t ld, SegBounds sb,
                const float *__restrict__ s_pos, const float *__restrict__ s_neg, int row_segments,
                int lo, int hi, uint8_t *__restrict__ c_pos, uint8_t *__restrict__ c_neg, int64_t ldc)
{
    __shared__ float sh_sp[kMaxBlocks];
    __shared__ float sh_sn[DUAL ? kMaxBlocks : 1];
    __shared__ int sh_kb[SQ_MAX_P + 1];
    const int Qs = row_segments ? sb.Q : 1;
    for (int i = threadIdx.x; i < sb.P * Qs; i += kThreads) {
        sh_sp[i] = s_pos[i];
        if (DUAL) sh_sn[i] = s_neg[i];
    }
    for (int i = threadIdx.x; i <= sb.P; i += kThreads) sh_kb[i] = sb.kb[i];
    __syncthreads();

    const int V = (K + kVec - 1) / kVec;
    const int64_t idx = int64_t(blockIdx.x) * kThreads + threadIdx.x;
    if (idx >= M * int64_t(V)) return;
    const int64_t row = idx / V;
    const int k0 = int(idx - row * V) * kVec;

    int q = 0;
    if (row_segments) while (q + 1 < sb.Q && row >= sb.nb[q + 1]) q++;
    int p = 0;
    while (p + 1 < sb.P && k0 >= sh_kb[p + 1]) p++;

    const Tin *src = X + row * ld + k0;
    uint8_t *dp = c_pos + row * ldc + k0;
    uint8_t *dn = DUAL ? c_neg + row * ldc + k0 : nullptr;

    if (k0 + kVec <= sh_kb[p + 1]) {            // whole vector inside one K-segment (and inside K)
        const float sp = sh_sp[p * Qs + q];
        const float sn = DUAL ? sh_sn[p * Qs + q] : 0.0f;
        float x[kVec];
        load16(src, x);
        uint32_t wp[4] = {0, 0, 0, 0}, wn[4] = {0, 0, 0, 0};
#pragma unroll
        for (int i = 0; i < kVec; i++) {
            uint32_t a, b;
            quant1<CODE, DUAL>(x[i], sp, sn, lo, hi, a, b);
            wp[i >> 2] |= a << (8 * (i & 3));
            if (DUAL) wn[i >> 2] |= b << (8 * (i & 3));
        }
        *reinterpret_cast<uint4 *>(dp) = make_uint4(wp[0], wp[1], wp[2], wp[3]);
        if (DUAL) *reinterpret_cast<uint4 *>(dn) = make_uint4(wn[0], wn[1], wn[2], wn[3]);
    } else {                                    // vector crosses a segment bound or the end of the row
        const int n = min(kVec, K - k0);
        for (int i = 0; i < n; i++) {
            while (p + 1 < sb.P && k0 + i >= sh_kb[p + 1]) p++;
            uint32_t a, b;
            quant1<CODE, DUAL>(load1(src + i), sh_sp[p * Qs + q], DUAL ? sh_sn[p * Qs + q] : 0.0f, lo, hi, a, b);
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
    if (s_neg)
        quantize_kernel<Tin, CODE, true><<<unsigned(blocks), kThreads, 0, st>>>(
            X, M, int(K), ld, sb, s_pos, s_neg, row_segments, lo, hi, static_cast<uint8_t *>(c_pos),
            static_cast<uint8_t *>(c_neg), ldc);
    else
        quantize_kernel<Tin, CODE, false><<<unsigned(blocks), kThreads, 0, st>>>(
            X, M, int(K), ld, sb, s_pos, nullptr, row_segments, lo, hi, static_cast<uint8_t *>(c_pos),
            nullptr, ldc);
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
