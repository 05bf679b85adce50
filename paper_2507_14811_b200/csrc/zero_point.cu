// Offline fold of the zero-point term (App. A asymmetric recovery).  With symmetric weight codes the correction
//   - s_X s_W z_X rowsum(W^)      (the paper's W is k x n: the sum runs over the input dimension)
// does not depend on the token, so it is added to the bias once:
//   bias'[n] = bias[n] - sum_p s_x[p] s_w[p][q(n)] z_x[p] wsum[p][n],   wsum[p][n] = sum_{k in segment p} W^[n][k],
// after which the layer runs through the ordinary single-scale GEMM.  One warp per output channel; the sums are
// exact integers, the fold is one fp32 product per factor pair and one FMA per K-segment in ascending order.
#include "sq_common.cuh"

namespace sq {
namespace {

constexpr int kWarpsPerBlock = 8;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
fold_zero_point_kernel(const int8_t *__restrict__ Wq, int64_t ldw, int N, const SegBounds sb,
                       const float *__restrict__ s_x, const int32_t *__restrict__ z_x,
                       const float *__restrict__ s_w, const float *__restrict__ bias, float *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int n = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (n >= N) return;                                   // warp-uniform
    int q = 0;
    while (q + 1 < sb.Q && n >= sb.nb[q + 1]) q++;
    const int8_t *row = Wq + int64_t(n) * ldw;
    float v = bias ? bias[n] : 0.0f;
    for (int p = 0; p < sb.P; p++) {
        int sum = 0;                                      // |sum| <= 128 * 131072 < 2^31
        const int k_lo = sb.kb[p], k_hi = sb.kb[p + 1];
        // whole 32-bit words where the segment allows (rows are 16-byte aligned), single codes at its ends
        const int w_lo = (k_lo + 3) & ~3, w_hi = k_hi & ~3;
        if (w_lo <= w_hi) {
            for (int k = k_lo + lane; k < w_lo; k += 32) sum += row[k];
            for (int k = w_lo + 4 * lane; k < w_hi; k += 128)
                sum = __dp4a(*reinterpret_cast<const int *>(row + k), 0x01010101, sum);
            for (int k = w_hi + lane; k < k_hi; k += 32) sum += row[k];
        } else {
            for (int k = k_lo + lane; k < k_hi; k += 32) sum += row[k];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        const float c = __fmul_rn(s_x[p], s_w[p * sb.Q + q]);
        v = __fmaf_rn(-c, __int2float_rn(z_x[p] * sum), v);   // |z * sum| <= 128 * 127 * 131072 < 2^31
    }
    if (lane == 0) out[n] = v;
}

}  // namespace

sq_status launch_fold_zero_point(const void *Wq, int64_t ldw, int64_t N, int64_t K, const SegBounds &sb,
                                 const float *s_x, const int32_t *z_x, const float *s_w, const float *bias,
                                 float *bias_folded, cudaStream_t st)
{
    (void)K;
    const int64_t blocks = (N + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > 0x7FFFFFFF) return SQ_ERR_SHAPE;
    fold_zero_point_kernel<<<unsigned(blocks), kWarpsPerBlock * 32, 0, st>>>(static_cast<const int8_t *>(Wq), ldw, int(N),
                                                                            sb, s_x, z_x, s_w, bias, bias_folded);
    count_launch();
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { note_cuda_error(e); return SQ_ERR_CUDA; }
    return SQ_OK;
}

}  // namespace sq
