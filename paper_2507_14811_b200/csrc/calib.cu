// Min/max calibration (Sec. 4.3.2 scale formula; strict min/max, App. B sensitivity analysis):
// per K-segment extrema of a calibration batch, or per (K-segment, N-segment) abs-max of a weight
// matrix, reduced through ordered-integer atomics into workspace partials, then one IEEE division
// per scale.
#include <cuda_bf16.h>
#include <mutex>
#include "sq_common.cuh"

namespace sq {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerBlock = 64;

// monotone map float -> uint32 (a < b  <=>  enc(a) < enc(b)); 0 and 0xFFFFFFFF are never produced
// by finite inputs and serve as the "nothing seen" marks of the max / min slots.
__device__ __forceinline__ uint32_t enc(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float dec(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u);
}

__device__ __forceinline__ float ld1(const float *p) { return __ldg(p); }
__device__ __forceinline__ float ld1(const __nv_bfloat16 *p)
{
    return __uint_as_float(uint32_t(__ldg(reinterpret_cast<const unsigned short *>(p))) << 16);
}

__global__ void calib_init_kernel(uint32_t *partials, int nblocks)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nblocks) { partials[2 * i] = 0u; partials[2 * i + 1] = 0xFFFFFFFFu; }
}

// grid.y covers columns (one column per thread), grid.x covers chunks of kRowsPerBlock rows.
// Consecutive threads read consecutive columns of the same row: coalesced.
template <typename Tin>
__global__ void __launch_bounds__(kThreads)
calib_reduce_kernel(const Tin *__restrict__ X, int64_t rows, int K, int64_t ld, SegBounds sb, int is_weight,
                    uint32_t *__restrict__ partials)
{
    __shared__ uint32_t sh_max[kMaxBlocks];
    __shared__ uint32_t sh_min[kMaxBlocks];
    const int Qs = is_weight ? sb.Q : 1;
    const int nblk = sb.P * Qs;
    for (int i = threadIdx.x; i < nblk; i += kThreads) { sh_max[i] = 0u; sh_min[i] = 0xFFFFFFFFu; }
    __syncthreads();

    const int k = blockIdx.y * kThreads + threadIdx.x;
    const int64_t r0 = int64_t(blockIdx.x) * kRowsPerBlock;
    const int64_t r1 = min(rows, r0 + kRowsPerBlock);
    if (k < K && r0 < r1) {
        int p = 0;
        while (p + 1 < sb.P && k >= sb.kb[p + 1]) p++;
        int q = 0;
        if (is_weight) while (q + 1 < sb.Q && r0 >= sb.nb[q + 1]) q++;
        float mx = -INFINITY, mn = INFINITY;
        for (int64_t r = r0; r < r1; r++) {
            if (is_weight && q + 1 < sb.Q && r >= sb.nb[q + 1]) {       // row enters the next N-segment
                atomicMax(&sh_max[p * Qs + q], enc(mx));
                atomicMin(&sh_min[p * Qs + q], enc(mn));
                mx = -INFINITY; mn = INFINITY;
                while (q + 1 < sb.Q && r >= sb.nb[q + 1]) q++;
            }
            float x = ld1(X + r * ld + k);
            mx = fmaxf(mx, x);
            mn = fminf(mn, x);
        }
        atomicMax(&sh_max[p * Qs + q], enc(mx));
        atomicMin(&sh_min[p * Qs + q], enc(mn));
    }
    __syncthreads();
    for (int i = threadIdx.x; i < nblk; i += kThreads) {
        if (sh_max[i] != 0u) atomicMax(&partials[2 * i], sh_max[i]);
        if (sh_min[i] != 0xFFFFFFFFu) atomicMin(&partials[2 * i + 1], sh_min[i]);
    }
}

__global__ void calib_finalize_kernel(const uint32_t *__restrict__ partials, int nblocks, int is_weight, int dual,
                                      float q_max, float q_min_abs, float *__restrict__ s_pos,
                                      float *__restrict__ s_neg)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nblocks) return;
    const uint32_t emx = partials[2 * i], emn = partials[2 * i + 1];
    const float mx = (emx == 0u || emx == enc(-INFINITY)) ? 0.0f : dec(emx);
    const float mn = (emn == 0xFFFFFFFFu || emn == enc(INFINITY)) ? 0.0f : dec(emn);
    if (!is_weight && dual) {
        const float hi = fmaxf(mx, 0.0f), lo = fmaxf(-mn, 0.0f);
        s_pos[i] = hi > 0.0f ? __fdiv_rn(hi, q_max) : 1.0f;
        s_neg[i] = lo > 0.0f ? __fdiv_rn(lo, q_min_abs) : 1.0f;
    } else {
        const float a = fmaxf(fabsf(mx), fabsf(mn));
        s_pos[i] = a > 0.0f ? __fdiv_rn(a, q_max) : 1.0f;
    }
}

// App. A asymmetric quantizer: s = (hi - lo) / 255 and z = -128 - round(lo / s) from the extrema widened to
// contain 0 (one fp32 subtraction, two IEEE divisions, round half to even); a zero range gives s = 1, z = 0.
__global__ void calib_finalize_zero_point_kernel(const uint32_t *__restrict__ partials, int nblocks,
                                                 float *__restrict__ s_x, int32_t *__restrict__ z_x)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nblocks) return;
    const uint32_t emx = partials[2 * i], emn = partials[2 * i + 1];
    const float mx = (emx == 0u || emx == enc(-INFINITY)) ? 0.0f : dec(emx);
    const float mn = (emn == 0xFFFFFFFFu || emn == enc(INFINITY)) ? 0.0f : dec(emn);
    const float hi = fmaxf(mx, 0.0f), lo = fminf(mn, 0.0f);
    const float range = __fsub_rn(hi, lo);
    if (range > 0.0f) {
        const float s = __fdiv_rn(range, 255.0f);
        const float zf = __fsub_rn(-128.0f, rintf(__fdiv_rn(lo, s)));
        s_x[i] = s;
        z_x[i] = int(fminf(fmaxf(zf, -128.0f), 127.0f));
    } else {
        s_x[i] = 1.0f;
        z_x[i] = 0;
    }
}

// Launch shape of the reduction; false if the matrix is beyond what one grid covers (checked before any launch).
bool calib_grid(int64_t rows, int64_t K, dim3 *grid)
{
    const int64_t gx = (rows + kRowsPerBlock - 1) / kRowsPerBlock, gy = (K + kThreads - 1) / kThreads;
    if (gx < 1 || gy < 1 || gx > 0x7FFFFFFFll || gy > 65535) return false;
    *grid = dim3(unsigned(gx), unsigned(gy));
    return true;
}

void launch_reduce(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb, int is_weight,
                   int nblocks, uint32_t *partials, dim3 grid, cudaStream_t st)
{
    calib_init_kernel<<<(nblocks + 255) / 256, 256, 0, st>>>(partials, nblocks);
    if (dt == SQ_F32)
        calib_reduce_kernel<float><<<grid, kThreads, 0, st>>>(static_cast<const float *>(X), rows, int(K), ld, sb,
                                                              is_weight, partials);
    else
        calib_reduce_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(static_cast<const __nv_bfloat16 *>(X), rows,
                                                                      int(K), ld, sb, is_weight, partials);
}

}  // namespace

sq_status launch_calib(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                       int is_weight, int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                       uint32_t *partials, cudaStream_t st)
{
    const int nblocks = sb.P * (is_weight ? sb.Q : 1);
    dim3 grid;
    if (!calib_grid(rows, K, &grid)) return SQ_ERR_SHAPE;      // nothing has been launched yet
    launch_reduce(X, dt, rows, K, ld, sb, is_weight, nblocks, partials, grid, st);
    calib_finalize_kernel<<<(nblocks + 255) / 256, 256, 0, st>>>(partials, nblocks, is_weight, dual, q_max, q_min_abs,
                                                                 s_pos, s_neg);
    count_launch(3);
    return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

sq_status launch_calib_zero_point(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                                  float *s_x, int32_t *z_x, uint32_t *partials, cudaStream_t st)
{
    dim3 grid;
    if (!calib_grid(rows, K, &grid)) return SQ_ERR_SHAPE;
    launch_reduce(X, dt, rows, K, ld, sb, 0, sb.P, partials, grid, st);
    calib_finalize_zero_point_kernel<<<(sb.P + 255) / 256, 256, 0, st>>>(partials, sb.P, s_x, z_x);
    count_launch(3);
    return cudaGetLastError() == cudaSuccess ? SQ_OK : SQ_ERR_CUDA;
}

namespace {

// ----------------------------------------------------------------------------- built-in scratch
// Reduction partials for callers that have no device allocator to take a workspace from: 2 words per
// (K-segment, N-segment) block, SQ_STATIC_CALIB_MAX_BLOCKS blocks, 8 KiB.  The array lives in the
// library's device image, so every GPU that loads the library holds it until the process exits, and
// every call on that GPU shares it.
static __device__ __align__(256) uint32_t g_static_partials[SQ_STATIC_CALIB_MAX_BLOCKS * 2];

// In host code the name g_static_partials is only a handle for the runtime; the device address has
// to be asked for, once per device, with that device current.
static sq_status static_partials_address(uint32_t **out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static uint32_t *addr[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) return SQ_ERR_CUDA;
        addr[dev] = static_cast<uint32_t *>(p);
    }
    *out = addr[dev];
    return SQ_OK;
}

}  // namespace

sq_status launch_calib_static(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                              int is_weight, int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                              cudaStream_t st)
{
    if (sb.P * (is_weight ? sb.Q : 1) > SQ_STATIC_CALIB_MAX_BLOCKS) return SQ_ERR_UNSUPPORTED;
    uint32_t *partials = nullptr;
    const sq_status r = static_partials_address(&partials);
    if (r != SQ_OK) return r;
    // launch_calib's first kernel resets the partials it is going to use, so the previous call's
    // contents never leak into this one
    return launch_calib(X, dt, rows, K, ld, sb, is_weight, dual, q_max, q_min_abs, s_pos, s_neg, partials, st);
}

}  // namespace sq
