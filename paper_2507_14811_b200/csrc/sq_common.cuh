// Internal declarations shared by the CUDA translation units of the library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include "segquant.h"

namespace sq {

// Workspace layout (device, 256-byte aligned):
//   [0,256)        status words: word 0 = first expired wait (0 = none)
//   [256, 256+32Ki) calibration partials: 2 ordered-uint words per (p,q) block
constexpr size_t kWsStatusBytes = 256;
constexpr int kMaxBlocks = SQ_MAX_P * SQ_MAX_Q;               // 4096 (p,q) blocks
constexpr size_t kWsCalibBytes = size_t(kMaxBlocks) * 2 * 4;  // 32 KiB
constexpr size_t kWsBytes = kWsStatusBytes + kWsCalibBytes;

// Segment bounds by value in kernel parameters (constant bank).
struct SegBounds {
    int P, Q;
    int kb[SQ_MAX_P + 1];
    int nb[SQ_MAX_Q + 1];
};

struct HostSeg {
    SegBounds b;
    sq_status status;
};

// Validates a segment table against K and N and copies it (host side).
HostSeg load_segtable(const sq_segtable *seg, int64_t K, int64_t N);

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void count_launch(int n = 1);
void note_cuda_error(cudaError_t e);   // remembered for segquant_last_cuda_error()

// per-code ranges
inline float code_qmax(sq_code c) { return c == SQ_CODE_INT8 ? 127.0f : 448.0f; }
inline float code_qmin_abs(sq_code c, uint32_t flags)
{
    if (c == SQ_CODE_INT8) return (flags & SQ_FLAG_QMIN_SYM) ? 127.0f : 128.0f;
    return 448.0f;
}

// kernels' host launchers (defined in the .cu files)
sq_status launch_calib(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                       int is_weight, int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                       uint32_t *partials, cudaStream_t st);

sq_status launch_calib_static(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                              int is_weight, int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                              cudaStream_t st);

// Parameters of the quantize kernel (by value, constant bank).
struct QuantParams {
    const void *X;
    int64_t M;
    int K;
    int64_t ld;
    SegBounds sb;
    const float *s_pos, *s_neg;
    const int32_t *zp;        // zero-point mode: z per K-segment
    int row_segments;         // weights: the scale also depends on the row's N-segment
    int lo, hi;
    uint8_t *c_pos, *c_neg;
    int64_t ldc;
    int V, R;
    int act;                  // PRE: 0 = none, 1 = SiLU, 2 = GELU applied to the input first
    const float *mult;        // PRE: per-channel multiplier [K] applied after it, or nullptr
};

// A quantize launch worked out ahead of time.
struct QuantLaunch {
    QuantParams prm;
    const void *kernel;
    unsigned blocks;
    unsigned threads;         // 0: the kernel's default block size
    unsigned smem;            // dynamic shared memory
};

// zero_point != nullptr selects the App. A asymmetric quantizer (int8); act / mult: optional activation
// function (0 none, 1 SiLU, 2 GELU) and per-channel multiplier [K] applied in front of the quantizer
sq_status launch_quantize(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                          const float *s_pos, const float *s_neg, const int32_t *zero_point, int row_segments,
                          sq_code code, float q_max, float q_min_abs, int act, const float *mult,
                          void *c_pos, void *c_neg, int64_t ldc, cudaStream_t st);

sq_status prepare_quantize(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                           const float *s_pos, const float *s_neg, const int32_t *zero_point, int row_segments,
                           sq_code code, float q_max, float q_min_abs, int act, const float *mult,
                           void *c_pos, void *c_neg, int64_t ldc, QuantLaunch *out);    // launches nothing
sq_status run_quantize(const QuantLaunch &l, cudaStream_t st);                          // one launch, no queries
void set_quantize_table_mode(int mode);      // fused activation by table: 0 automatic, 1 wherever possible, 2 never (tests)

// One scale per (row, K-segment) from the row's own extrema, written to s_pos / s_neg [rows][P], and the int8 codes
// quantized with them (per-token activations, q_max 127; per-channel 4-bit weights, q_max 7).
sq_status launch_quantize_per_row(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld, const SegBounds &sb,
                                  int dual, float q_max, float q_min_abs, float *s_pos, float *s_neg,
                                  void *c_pos, void *c_neg, int64_t ldc, cudaStream_t st);
sq_status launch_pack_w4(const void *Wq8, int64_t ld8, int64_t N, int64_t K, void *Wq4, int64_t ld4, int unpack,
                         cudaStream_t st);

sq_status launch_calib_zero_point(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld, const SegBounds &sb,
                                  float *s_x, int32_t *z_x, uint32_t *partials, cudaStream_t st);

sq_status launch_fold_zero_point(const void *Wq, int64_t ldw, int64_t N, int64_t K, const SegBounds &sb,
                                 const float *s_x, const int32_t *z_x, const float *s_w, const float *bias,
                                 float *bias_folded, cudaStream_t st);

struct GemmArgs {
    const void *a_pos, *a_neg;   // code matrices [M,K]; a_neg == nullptr: single path
    int64_t lda;
    const void *b;               // weight codes [N,K]
    int64_t ldb;
    int64_t M, N, K;
    SegBounds sb;
    sq_code code;
    const float *s_pos, *s_neg, *s_w, *bias;
    const float *row_pos, *row_neg, *col_scale;   // W4A8: per-token and per-channel scales (then s_pos / s_neg / s_w unused)
    void *Y;
    sq_dtype y_dtype;
    int64_t ldy;
    void *acc_dump;
    uint32_t *status;
    void *sk_scratch;            // split tiles: zero-filled device scratch behind the workspace's fixed part, or nullptr
    size_t sk_bytes;
};
// Parameters of the GEMM kernel (by value, constant bank).
struct KernelParams {
    int M, N, K;
    int nacc;          // P * npol
    int acc_stages;    // 1 or 2 accumulator sets in TMEM
    int stages;        // shared-memory ring depth
    int num_m_tiles, num_n_tiles;
    SegBounds sb;
    const float *s_pos, *s_neg, *s_w, *bias;
    const float *row_pos, *row_neg, *col_scale;   // per-token [M][P] and per-channel [N][P] scales instead of the tables
    uint32_t col_tab_bytes;                       // shared memory for the tile's channel scales (0: read from global)
    void *Y;
    long long ldy;     // elements
    int y_is_f32;
    int y_wide;        // rows of Y are 32-byte aligned: 256-bit stores allowed
    void *acc_dump;
    uint32_t *status;
    uint32_t *sk_counters;       // split tiles: arrivals per (tile, CTA of the pair), zero between launches
    uint8_t *sk_slots;           // split tiles: per (pair, slot, CTA) one CTA's raw accumulators
    int sk_kblocks;              // split tiles: K-blocks per tile (0: tiles are not split)
};

// A GEMM launch worked out ahead of time: kernel instantiation, tensor maps, parameters, grid.
struct GemmLaunch {
    CUtensorMap ta, tn, tb, ty;
    KernelParams prm;
    const void *kernel;
    unsigned grid, cluster;
    size_t smem;
    int device;
};
sq_status prepare_gemm(const GemmArgs &g, GemmLaunch *out);    // launches nothing
sq_status run_gemm(const GemmLaunch &l, cudaStream_t st);      // one launch, no queries
sq_status launch_gemm(const GemmArgs &g, cudaStream_t st);     // prepare + run
void set_gemm_tuning(int tile_n, int stages, int cta_group, int segment_mode);
// bytes behind the workspace's fixed part that let prepare_gemm split tiles for an [M, N] output on the current device
size_t gemm_split_scratch_bytes(int64_t M, int64_t N, int dual);

}  // namespace sq
