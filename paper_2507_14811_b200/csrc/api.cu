// C ABI: host-side validation and dispatch.  Every argument error is reported before any launch.  A layer call
// can also be prepared once (segquant_plan_layer) and replayed as two bare launches (segquant_plan_run).
#include <atomic>
#include <cstring>
#include "sq_common.cuh"

namespace sq {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(uint64_t(n), std::memory_order_relaxed); }

static std::atomic<int> g_last_cuda_error{0};
void note_cuda_error(cudaError_t e) { g_last_cuda_error.store(int(e), std::memory_order_relaxed); }

HostSeg load_segtable(const sq_segtable *seg, int64_t K, int64_t N)
{
    HostSeg h{};
    h.status = SQ_OK;
    if (!seg || !seg->kb || !seg->nb) { h.status = SQ_ERR_NULL; return h; }
    if (seg->P < 1 || seg->Q < 1) { h.status = SQ_ERR_SEGTABLE; return h; }
    if (seg->P > SQ_MAX_P || seg->Q > SQ_MAX_Q) { h.status = SQ_ERR_UNSUPPORTED; return h; }
    h.b.P = seg->P;
    h.b.Q = seg->Q;
    for (int i = 0; i <= seg->P; i++) h.b.kb[i] = seg->kb[i];
    for (int i = 0; i <= seg->Q; i++) h.b.nb[i] = seg->nb[i];
    if (h.b.kb[0] != 0 || h.b.kb[seg->P] != K || h.b.nb[0] != 0 || h.b.nb[seg->Q] != N) {
        h.status = SQ_ERR_SEGTABLE;
        return h;
    }
    for (int i = 0; i < seg->P; i++)
        if (h.b.kb[i + 1] <= h.b.kb[i]) { h.status = SQ_ERR_SEGTABLE; return h; }
    for (int i = 0; i < seg->Q; i++)
        if (h.b.nb[i + 1] <= h.b.nb[i]) { h.status = SQ_ERR_SEGTABLE; return h; }
    return h;
}

static size_t dt_size(sq_dtype dt) { return dt == SQ_F32 ? 4 : 2; }
static bool valid_dt(sq_dtype dt) { return dt == SQ_F32 || dt == SQ_BF16; }
static bool valid_code(sq_code c) { return c == SQ_CODE_INT8 || c == SQ_CODE_E4M3; }
constexpr int64_t kMaxDim = 1 << 30;
constexpr int64_t kMaxK = 131072;   // int8: 131072 * 128 * 127 < 2^31

static sq_status check_ws(void *ws, size_t bytes)
{
    if (!ws || bytes < kWsBytes) return SQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return SQ_ERR_ALIGN;
    return SQ_OK;
}

static sq_status check_matrix(const void *p, int64_t rows, int64_t cols, int64_t ld, size_t elem)
{
    if (!p) return SQ_ERR_NULL;
    if (rows <= 0 || cols <= 0 || rows > kMaxDim || cols > kMaxDim || ld < cols) return SQ_ERR_SHAPE;
    if (!aligned16(p) || (size_t(ld) * elem) % 16 != 0) return SQ_ERR_ALIGN;
    return SQ_OK;
}

// Validation shared by the GEMM entry points and the plan; fills `g` when everything is in order.
static sq_status gemm_args(const void *a_pos, const void *a_neg, int dual, int64_t ldx, const void *Wq, int64_t ldw,
                           int64_t M, int64_t N, int64_t K, const sq_segtable *seg, sq_code code,
                           const float *s_pos, const float *s_neg, const float *s_w, const float *bias, void *Y,
                           sq_dtype y_dtype, int64_t ldy, void *acc_dump, void *workspace, size_t ws_bytes,
                           GemmArgs *out, int per_token = 0)
{
    if (!s_pos || !s_w || (dual && (!a_neg || !s_neg))) return SQ_ERR_NULL;
    if (!valid_code(code) || !valid_dt(y_dtype)) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    if ((st = check_matrix(a_pos, M, K, ldx, 1)) != SQ_OK) return st;
    if (dual && (st = check_matrix(a_neg, M, K, ldx, 1)) != SQ_OK) return st;
    if ((st = check_matrix(Wq, N, K, ldw, 1)) != SQ_OK) return st;
    if ((st = check_matrix(Y, M, N, ldy, dt_size(y_dtype))) != SQ_OK) return st;
    if (K > kMaxK) return SQ_ERR_SHAPE;
    if (K % 16 != 0 || N % 8 != 0) return SQ_ERR_ALIGN;
    if (acc_dump && !aligned16(acc_dump)) return SQ_ERR_ALIGN;
    HostSeg hs = load_segtable(seg, K, N);
    if (hs.status != SQ_OK) return hs.status;
    for (int p = 1; p < hs.b.P; p++)
        if (hs.b.kb[p] % 32 != 0) return SQ_ERR_ALIGN;
    if (hs.b.P * (dual ? 2 : 1) * hs.b.Q > 2048) return SQ_ERR_UNSUPPORTED;   // dequantization factors kept in shared memory
    if ((st = check_ws(workspace, ws_bytes)) != SQ_OK) return st;

    GemmArgs &g = *out;
    g = GemmArgs{};
    g.a_pos = a_pos; g.a_neg = dual ? a_neg : nullptr; g.lda = ldx;
    g.b = Wq; g.ldb = ldw;
    g.M = M; g.N = N; g.K = K;
    g.sb = hs.b;
    g.code = code;
    if (per_token) {     // s_pos / s_neg are [M][P] token scales, s_w is [N][P] channel scales
        g.row_pos = s_pos; g.row_neg = dual ? s_neg : nullptr; g.col_scale = s_w;
    } else {
        g.s_pos = s_pos; g.s_neg = dual ? s_neg : nullptr; g.s_w = s_w;
    }
    g.bias = bias;
    g.Y = Y; g.y_dtype = y_dtype; g.ldy = ldy;
    g.acc_dump = acc_dump;
    g.status = static_cast<uint32_t *>(workspace);
    if (ws_bytes > kWsBytes) {           // a larger workspace: room for the partial sums of split tiles
        g.sk_scratch = static_cast<uint8_t *>(workspace) + kWsBytes;
        g.sk_bytes = ws_bytes - kWsBytes;
    }
    return SQ_OK;
}

static sq_status gemm_common(const void *a_pos, const void *a_neg, int dual, int64_t ldx, const void *Wq, int64_t ldw,
                             int64_t M, int64_t N, int64_t K, const sq_segtable *seg, sq_code code,
                             const float *s_pos, const float *s_neg, const float *s_w, const float *bias, void *Y,
                             sq_dtype y_dtype, int64_t ldy, void *acc_dump, void *workspace, size_t ws_bytes,
                             void *stream)
{
    GemmArgs g;
    const sq_status st = gemm_args(a_pos, a_neg, dual, ldx, Wq, ldw, M, N, K, seg, code, s_pos, s_neg, s_w, bias, Y,
                                   y_dtype, ldy, acc_dump, workspace, ws_bytes, &g);
    return st == SQ_OK ? launch_gemm(g, static_cast<cudaStream_t>(stream)) : st;
}

// What an sq_plan holds (copied in and out of the caller's storage, which need not be aligned for it).
struct LayerPlan {
    uint64_t magic;
    QuantLaunch quant;
    GemmLaunch gemm;
};
constexpr uint64_t kPlanMagic = 0x53514C41594552ull;   // "SQLAYER"
static_assert(sizeof(LayerPlan) <= sizeof(sq_plan), "sq_plan is too small for a layer plan");

}  // namespace sq

using namespace sq;

extern "C" {

size_t segquant_workspace_bytes(void) { return kWsBytes; }

size_t segquant_split_workspace_bytes(int64_t M, int64_t N, int dual)
{
    const size_t extra = gemm_split_scratch_bytes(M, N, dual);
    return extra ? kWsBytes + extra : 0;
}

sq_status segquant_calib_scales(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                const sq_segtable *seg, sq_code code, int is_weight, int dual, uint32_t flags,
                                float *s_pos, float *s_neg, void *workspace, size_t ws_bytes, void *stream)
{
    if (!s_pos || (!is_weight && dual && !s_neg)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    sq_status st = check_matrix(X, rows, K, ld, dt_size(dt));
    if (st != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, is_weight ? rows : (seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0));
    if (hs.status != SQ_OK) return hs.status;
    if ((st = check_ws(workspace, ws_bytes)) != SQ_OK) return st;
    uint32_t *partials = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + kWsStatusBytes);
    return launch_calib(X, dt, rows, K, ld, hs.b, is_weight, dual, code_qmax(code), code_qmin_abs(code, flags),
                        s_pos, s_neg, partials, static_cast<cudaStream_t>(stream));
}

sq_status segquant_calib_scales_static(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                       const sq_segtable *seg, sq_code code, int is_weight, int dual,
                                       uint32_t flags, float *s_pos, float *s_neg, void *stream)
{
    if (!s_pos || (!is_weight && dual && !s_neg)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    sq_status st = check_matrix(X, rows, K, ld, dt_size(dt));
    if (st != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, is_weight ? rows : (seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0));
    if (hs.status != SQ_OK) return hs.status;
    if (hs.b.P * (is_weight ? hs.b.Q : 1) > SQ_STATIC_CALIB_MAX_BLOCKS) return SQ_ERR_UNSUPPORTED;
    return launch_calib_static(X, dt, rows, K, ld, hs.b, is_weight, dual, code_qmax(code), code_qmin_abs(code, flags),
                               s_pos, s_neg, static_cast<cudaStream_t>(stream));
}

sq_status segquant_quantize_act(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                const sq_segtable *seg, const float *s_pos, const float *s_neg, sq_code code,
                                uint32_t flags, void *c_pos, void *c_neg, int64_t ldc, void *stream)
{
    if (!s_pos || (s_neg && !c_neg)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    if ((st = check_matrix(X, M, K, ld, dt_size(dt))) != SQ_OK) return st;
    if ((st = check_matrix(c_pos, M, K, ldc, 1)) != SQ_OK) return st;
    if (s_neg && (st = check_matrix(c_neg, M, K, ldc, 1)) != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0);
    if (hs.status != SQ_OK) return hs.status;
    return launch_quantize(X, dt, M, K, ld, hs.b, s_pos, s_neg, nullptr, 0, code, code_qmax(code),
                           code_qmin_abs(code, flags), 0, nullptr, c_pos, c_neg, ldc, static_cast<cudaStream_t>(stream));
}

sq_status segquant_quantize_act_fused(const void *H, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                      const sq_segtable *seg, const float *s_pos, const float *s_neg, sq_code code,
                                      uint32_t flags, sq_act act, const float *mult, void *c_pos, void *c_neg,
                                      int64_t ldc, void *stream)
{
    if (!s_pos || (s_neg && !c_neg)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    if (act != SQ_ACT_NONE && act != SQ_ACT_SILU && act != SQ_ACT_GELU && act != SQ_ACT_GEGLU) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    const bool gated = act == SQ_ACT_GEGLU;                  // the row holds 2 K pre-activations: value half, gate half
    if (gated && K > 0 && (K * int64_t(dt_size(dt))) % 16 != 0) return SQ_ERR_ALIGN;
    if ((st = check_matrix(H, M, gated ? 2 * K : K, ld, dt_size(dt))) != SQ_OK) return st;
    if ((st = check_matrix(c_pos, M, K, ldc, 1)) != SQ_OK) return st;
    if (s_neg && (st = check_matrix(c_neg, M, K, ldc, 1)) != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0);
    if (hs.status != SQ_OK) return hs.status;
    return launch_quantize(H, dt, M, K, ld, hs.b, s_pos, s_neg, nullptr, 0, code, code_qmax(code),
                           code_qmin_abs(code, flags), int(act), mult, c_pos, c_neg, ldc,
                           static_cast<cudaStream_t>(stream));
}

sq_status segquant_calib_zero_point(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                    const sq_segtable *seg, float *s_x, int32_t *z_x, void *workspace,
                                    size_t ws_bytes, void *stream)
{
    if (!s_x || !z_x) return SQ_ERR_NULL;
    if (!valid_dt(dt)) return SQ_ERR_UNSUPPORTED;
    sq_status st = check_matrix(X, rows, K, ld, dt_size(dt));
    if (st != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0);
    if (hs.status != SQ_OK) return hs.status;
    if ((st = check_ws(workspace, ws_bytes)) != SQ_OK) return st;
    uint32_t *partials = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + kWsStatusBytes);
    return launch_calib_zero_point(X, dt, rows, K, ld, hs.b, s_x, z_x, partials, static_cast<cudaStream_t>(stream));
}

sq_status segquant_quantize_act_zero_point(const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                           const sq_segtable *seg, const float *s_x, const int32_t *z_x,
                                           void *codes, int64_t ldc, void *stream)
{
    if (!s_x || !z_x) return SQ_ERR_NULL;
    if (!valid_dt(dt)) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    if ((st = check_matrix(X, M, K, ld, dt_size(dt))) != SQ_OK) return st;
    if ((st = check_matrix(codes, M, K, ldc, 1)) != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0);
    if (hs.status != SQ_OK) return hs.status;
    return launch_quantize(X, dt, M, K, ld, hs.b, s_x, nullptr, z_x, 0, SQ_CODE_INT8, 127.0f, 128.0f, 0, nullptr, codes,
                           nullptr, ldc, static_cast<cudaStream_t>(stream));
}

sq_status segquant_fold_zero_point(const void *Wq, int64_t ldw, int64_t N, int64_t K, const sq_segtable *seg,
                                   const float *s_x, const int32_t *z_x, const float *s_w, const float *bias,
                                   float *bias_folded, void *stream)
{
    if (!s_x || !z_x || !s_w || !bias_folded) return SQ_ERR_NULL;
    sq_status st;
    if ((st = check_matrix(Wq, N, K, ldw, 1)) != SQ_OK) return st;
    if (K > kMaxK) return SQ_ERR_SHAPE;
    HostSeg hs = load_segtable(seg, K, N);
    if (hs.status != SQ_OK) return hs.status;
    return launch_fold_zero_point(Wq, ldw, N, K, hs.b, s_x, z_x, s_w, bias, bias_folded,
                                  static_cast<cudaStream_t>(stream));
}

sq_status segquant_quantize_weight(const void *W, sq_dtype dt, int64_t N, int64_t K, int64_t ld,
                                   const sq_segtable *seg, const float *s_w, sq_code code, uint32_t flags,
                                   void *Wq, int64_t ldq, void *stream)
{
    (void)flags;
    if (!s_w) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    if ((st = check_matrix(W, N, K, ld, dt_size(dt))) != SQ_OK) return st;
    if ((st = check_matrix(Wq, N, K, ldq, 1)) != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, N);
    if (hs.status != SQ_OK) return hs.status;
    return launch_quantize(W, dt, N, K, ld, hs.b, s_w, nullptr, nullptr, 1, code, code_qmax(code), code_qmax(code), 0,
                           nullptr, Wq, nullptr, ldq, static_cast<cudaStream_t>(stream));
}

sq_status segquant_seglinear_gemm(const void *Xq, int64_t ldx, const void *Wq, int64_t ldw, int64_t M, int64_t N,
                                  int64_t K, const sq_segtable *seg, sq_code code, const float *s_x,
                                  const float *s_w, const float *bias, void *Y, sq_dtype y_dtype, int64_t ldy,
                                  void *acc_dump, void *workspace, size_t ws_bytes, void *stream)
{
    return gemm_common(Xq, nullptr, 0, ldx, Wq, ldw, M, N, K, seg, code, s_x, nullptr, s_w, bias, Y, y_dtype, ldy,
                       acc_dump, workspace, ws_bytes, stream);
}

sq_status segquant_dualscale_gemm(const void *Xq_pos, const void *Xq_neg, int64_t ldx, const void *Wq, int64_t ldw,
                                  int64_t M, int64_t N, int64_t K, const sq_segtable *seg, sq_code code,
                                  const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                                  void *Y, sq_dtype y_dtype, int64_t ldy, void *acc_dump, void *workspace,
                                  size_t ws_bytes, void *stream)
{
    return gemm_common(Xq_pos, Xq_neg, 1, ldx, Wq, ldw, M, N, K, seg, code, s_pos, s_neg, s_w, bias, Y, y_dtype,
                       ldy, acc_dump, workspace, ws_bytes, stream);
}

size_t segquant_layer_scratch_bytes(int64_t M, int64_t K, int dual)
{
    if (M <= 0 || K <= 0) return 0;
    const size_t ldc = (size_t(K) + 127) & ~size_t(127);
    const size_t one = (size_t(M) * ldc + 255) & ~size_t(255);
    return one * (dual ? 2 : 1);
}

sq_status segquant_layer_forward(const void *X, int x_on_host, void *x_stage, sq_dtype dt, int64_t M, int64_t K,
                                 int64_t ld, const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg,
                                 sq_code code, const float *s_pos, const float *s_neg, const float *s_w,
                                 const float *bias, uint32_t flags, void *Y, int y_on_host, void *y_stage,
                                 sq_dtype y_dtype, int64_t ldy, void *scratch, size_t scratch_bytes,
                                 void *workspace, size_t ws_bytes, void *stream)
{
    if (!X || !Y || !scratch || (x_on_host && !x_stage) || (y_on_host && !y_stage)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_dt(y_dtype)) return SQ_ERR_UNSUPPORTED;
    if (M <= 0 || K <= 0 || N <= 0 || ld < K || ldy < N) return SQ_ERR_SHAPE;
    const int dual = s_neg != nullptr;
    if (scratch_bytes < segquant_layer_scratch_bytes(M, K, dual)) return SQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return SQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const void *xd = X;
    if (x_on_host) {
        if (cudaMemcpyAsync(x_stage, X, size_t(M) * ld * dt_size(dt), cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SQ_ERR_CUDA;
        xd = x_stage;
    }
    const int64_t ldc = (K + 127) & ~int64_t(127);
    uint8_t *c_pos = static_cast<uint8_t *>(scratch);
    uint8_t *c_neg = dual ? c_pos + ((size_t(M) * ldc + 255) & ~size_t(255)) : nullptr;
    sq_status r = segquant_quantize_act(xd, dt, M, K, ld, seg, s_pos, s_neg, code, flags, c_pos, c_neg, ldc, stream);
    if (r != SQ_OK) return r;
    void *yd = y_on_host ? y_stage : Y;
    r = dual ? segquant_dualscale_gemm(c_pos, c_neg, ldc, Wq, ldw, M, N, K, seg, code, s_pos, s_neg, s_w, bias, yd,
                                       y_dtype, ldy, nullptr, workspace, ws_bytes, stream)
             : segquant_seglinear_gemm(c_pos, ldc, Wq, ldw, M, N, K, seg, code, s_pos, s_w, bias, yd, y_dtype, ldy,
                                       nullptr, workspace, ws_bytes, stream);
    if (r != SQ_OK) return r;
    if (y_on_host &&
        cudaMemcpyAsync(Y, y_stage, size_t(M) * ldy * dt_size(y_dtype), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return SQ_ERR_CUDA;
    return SQ_OK;
}

sq_status segquant_layer_forward_pipelined(const void *X, void *x_stage, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                                           const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg,
                                           sq_code code, const float *s_pos, const float *s_neg, const float *s_w,
                                           const float *bias, uint32_t flags, void *Y, void *y_stage,
                                           sq_dtype y_dtype, int64_t ldy, void *scratch, size_t scratch_bytes,
                                           void *workspace, size_t ws_bytes, int chunks, void *stream,
                                           void *stream_in, void *stream_out)
{
    if (!X || !Y || !scratch || !x_stage || !y_stage) return SQ_ERR_NULL;
    if (!valid_dt(dt) || !valid_dt(y_dtype)) return SQ_ERR_UNSUPPORTED;
    if (M <= 0 || K <= 0 || N <= 0 || ld < K || ldy < N || chunks < 1 || chunks > 64) return SQ_ERR_SHAPE;
    if (stream_in == stream || stream_out == stream || stream_in == stream_out) return SQ_ERR_UNSUPPORTED;
    const int dual = s_neg != nullptr;
    if (scratch_bytes < segquant_layer_scratch_bytes(M, K, dual)) return SQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return SQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream), sin = static_cast<cudaStream_t>(stream_in),
                 sout = static_cast<cudaStream_t>(stream_out);
    const int64_t ldc = (K + 127) & ~int64_t(127);
    uint8_t *c_pos = static_cast<uint8_t *>(scratch);
    uint8_t *c_neg = dual ? c_pos + ((size_t(M) * ldc + 255) & ~size_t(255)) : nullptr;
    // rows per chunk: whole 256-row tiles
    int64_t rows = ((M + chunks - 1) / chunks + 255) & ~int64_t(255);

    // events order the three streams; they are created for this call and released when their work is done
    cudaEvent_t ev[2 * 64 + 2];
    int nev = 0;
    auto new_event = [&]() -> cudaEvent_t {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        ev[nev++] = e;
        return e;
    };
    sq_status r = SQ_OK;
    auto fail = [&](sq_status code_) { if (r == SQ_OK) r = code_; };
    cudaEvent_t e0 = new_event();       // the staging buffers may still be in use by earlier work on `stream`
    if (!e0 || cudaEventRecord(e0, st) != cudaSuccess || cudaStreamWaitEvent(sin, e0, 0) != cudaSuccess ||
        cudaStreamWaitEvent(sout, e0, 0) != cudaSuccess)
        fail(SQ_ERR_CUDA);
    cudaEvent_t last_out = nullptr;
    for (int64_t r0 = 0; r0 < M && r == SQ_OK; r0 += rows) {
        const int64_t m = r0 + rows <= M ? rows : M - r0;
        const size_t x_off = size_t(r0) * ld * dt_size(dt), y_off = size_t(r0) * ldy * dt_size(y_dtype);
        cudaEvent_t e_in = new_event(), e_done = new_event();
        if (!e_in || !e_done) { fail(SQ_ERR_CUDA); break; }
        if (cudaMemcpyAsync(static_cast<uint8_t *>(x_stage) + x_off, static_cast<const uint8_t *>(X) + x_off,
                            size_t(m) * ld * dt_size(dt), cudaMemcpyHostToDevice, sin) != cudaSuccess ||
            cudaEventRecord(e_in, sin) != cudaSuccess || cudaStreamWaitEvent(st, e_in, 0) != cudaSuccess) {
            fail(SQ_ERR_CUDA);
            break;
        }
        sq_status q = segquant_quantize_act(static_cast<uint8_t *>(x_stage) + x_off, dt, m, K, ld, seg, s_pos, s_neg, code,
                                            flags, c_pos + size_t(r0) * ldc, dual ? c_neg + size_t(r0) * ldc : nullptr,
                                            ldc, stream);
        if (q == SQ_OK)
            q = dual ? segquant_dualscale_gemm(c_pos + size_t(r0) * ldc, c_neg + size_t(r0) * ldc, ldc, Wq, ldw, m, N, K,
                                               seg, code, s_pos, s_neg, s_w, bias, static_cast<uint8_t *>(y_stage) + y_off,
                                               y_dtype, ldy, nullptr, workspace, ws_bytes, stream)
                     : segquant_seglinear_gemm(c_pos + size_t(r0) * ldc, ldc, Wq, ldw, m, N, K, seg, code, s_pos, s_w, bias,
                                               static_cast<uint8_t *>(y_stage) + y_off, y_dtype, ldy, nullptr, workspace,
                                               ws_bytes, stream);
        if (q != SQ_OK) { fail(q); break; }
        if (cudaEventRecord(e_done, st) != cudaSuccess || cudaStreamWaitEvent(sout, e_done, 0) != cudaSuccess ||
            cudaMemcpyAsync(static_cast<uint8_t *>(Y) + y_off, static_cast<uint8_t *>(y_stage) + y_off,
                            size_t(m) * ldy * dt_size(y_dtype), cudaMemcpyDeviceToHost, sout) != cudaSuccess) {
            fail(SQ_ERR_CUDA);
            break;
        }
    }
    // `stream` completes only when the last output copy has: the caller synchronizes one stream
    last_out = new_event();
    if (!last_out || cudaEventRecord(last_out, sout) != cudaSuccess || cudaStreamWaitEvent(st, last_out, 0) != cudaSuccess)
        fail(SQ_ERR_CUDA);
    for (int i = 0; i < nev; i++) cudaEventDestroy(ev[i]);
    return r;
}

sq_status segquant_quantize_per_row(const void *X, sq_dtype dt, int64_t rows, int64_t K, int64_t ld,
                                    const sq_segtable *seg, int bits, uint32_t flags, float *s_pos, float *s_neg,
                                    void *c_pos, void *c_neg, int64_t ldc, void *stream)
{
    if (!s_pos || (s_neg && !c_neg)) return SQ_ERR_NULL;
    if (!valid_dt(dt) || (bits != 8 && bits != 4) || (bits == 4 && s_neg)) return SQ_ERR_UNSUPPORTED;
    sq_status st;
    if ((st = check_matrix(X, rows, K, ld, dt_size(dt))) != SQ_OK) return st;
    if ((st = check_matrix(c_pos, rows, K, ldc, 1)) != SQ_OK) return st;
    if (s_neg && (st = check_matrix(c_neg, rows, K, ldc, 1)) != SQ_OK) return st;
    HostSeg hs = load_segtable(seg, K, seg && seg->nb && seg->Q >= 1 ? seg->nb[seg->Q] : 0);
    if (hs.status != SQ_OK) return hs.status;
    const float q_max = bits == 4 ? 7.0f : 127.0f;
    const float q_min_abs = bits == 4 ? 7.0f : code_qmin_abs(SQ_CODE_INT8, flags);
    return launch_quantize_per_row(X, dt, rows, K, ld, hs.b, s_neg != nullptr, q_max, q_min_abs, s_pos, s_neg, c_pos,
                                   c_neg, ldc, static_cast<cudaStream_t>(stream));
}

static sq_status w4_common(const void *w8, int64_t ld8, void *w4, int64_t ld4, int64_t N, int64_t K, int unpack, void *stream)
{
    sq_status st;
    if ((st = check_matrix(w8, N, K, ld8, 1)) != SQ_OK) return st;
    if (K % 16 != 0) return SQ_ERR_ALIGN;
    if (!w4) return SQ_ERR_NULL;
    if (ld4 < K / 2) return SQ_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(w4) & 7u) || ld4 % 8 != 0) return SQ_ERR_ALIGN;
    return launch_pack_w4(w8, ld8, N, K, w4, ld4, unpack, static_cast<cudaStream_t>(stream));
}

sq_status segquant_pack_w4(const void *Wq8, int64_t ld8, int64_t N, int64_t K, void *Wq4, int64_t ld4, void *stream)
{
    return w4_common(Wq8, ld8, Wq4, ld4, N, K, 0, stream);
}

sq_status segquant_unpack_w4(const void *Wq4, int64_t ld4, int64_t N, int64_t K, void *Wq8, int64_t ld8, void *stream)
{
    return w4_common(Wq8, ld8, const_cast<void *>(Wq4), ld4, N, K, 1, stream);
}

sq_status segquant_w4a8_gemm(const void *Xq_pos, const void *Xq_neg, int64_t ldx, const void *Wq8, int64_t ldw,
                             int64_t M, int64_t N, int64_t K, const sq_segtable *seg, const float *s_pos,
                             const float *s_neg, const float *s_w, const float *bias, void *Y, sq_dtype y_dtype,
                             int64_t ldy, void *acc_dump, void *workspace, size_t ws_bytes, void *stream)
{
    const int dual = Xq_neg != nullptr;
    if (seg && seg->Q != 1) return SQ_ERR_SEGTABLE;             // per-channel scales subsume output segments
    GemmArgs g;
    const sq_status st = gemm_args(Xq_pos, Xq_neg, dual, ldx, Wq8, ldw, M, N, K, seg, SQ_CODE_INT8, s_pos, s_neg, s_w,
                                   bias, Y, y_dtype, ldy, acc_dump, workspace, ws_bytes, &g, 1);
    return st == SQ_OK ? launch_gemm(g, static_cast<cudaStream_t>(stream)) : st;
}

sq_status segquant_plan_layer(sq_plan *plan, const void *X, sq_dtype dt, int64_t M, int64_t K, int64_t ld,
                              const void *Wq, int64_t ldw, int64_t N, const sq_segtable *seg, sq_code code,
                              const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                              uint32_t flags, void *Y, sq_dtype y_dtype, int64_t ldy, void *scratch,
                              size_t scratch_bytes, void *workspace, size_t ws_bytes)
{
    if (!plan || !X || !Y || !scratch || !s_pos) return SQ_ERR_NULL;
    std::memset(plan, 0, sizeof(*plan));
    if (!valid_dt(dt) || !valid_dt(y_dtype) || !valid_code(code)) return SQ_ERR_UNSUPPORTED;
    const int dual = s_neg != nullptr;
    sq_status st;
    if ((st = check_matrix(X, M, K, ld, dt_size(dt))) != SQ_OK) return st;
    if (scratch_bytes < segquant_layer_scratch_bytes(M, K, dual)) return SQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(scratch) & 255u) return SQ_ERR_ALIGN;
    const int64_t ldc = (K + 127) & ~int64_t(127);
    uint8_t *c_pos = static_cast<uint8_t *>(scratch);
    uint8_t *c_neg = dual ? c_pos + ((size_t(M) * ldc + 255) & ~size_t(255)) : nullptr;
    GemmArgs g;
    if ((st = gemm_args(c_pos, c_neg, dual, ldc, Wq, ldw, M, N, K, seg, code, s_pos, s_neg, s_w, bias, Y, y_dtype, ldy,
                        nullptr, workspace, ws_bytes, &g)) != SQ_OK)
        return st;
    LayerPlan lp{};
    if ((st = prepare_quantize(X, dt, M, K, ld, g.sb, s_pos, s_neg, nullptr, 0, code, code_qmax(code),
                               code_qmin_abs(code, flags), 0, nullptr, c_pos, c_neg, ldc, &lp.quant)) != SQ_OK)
        return st;
    if ((st = prepare_gemm(g, &lp.gemm)) != SQ_OK) return st;
    lp.magic = kPlanMagic;
    std::memcpy(plan, &lp, sizeof(lp));
    return SQ_OK;
}

sq_status segquant_plan_run(const sq_plan *plan, void *stream)
{
    if (!plan) return SQ_ERR_NULL;
    LayerPlan lp;
    std::memcpy(&lp, plan, sizeof(lp));
    if (lp.magic != kPlanMagic) return SQ_ERR_UNSUPPORTED;     // never built, or a failed segquant_plan_layer
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SQ_ERR_CUDA;
    if (dev != lp.gemm.device) return SQ_ERR_UNSUPPORTED;      // plans belong to the device they were built on
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const sq_status r = run_quantize(lp.quant, st);
    return r == SQ_OK ? run_gemm(lp.gemm, st) : r;
}

sq_status segquant_last_device_status(void *workspace, void *stream, uint32_t *detail)
{
    if (!workspace) return SQ_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SQ_ERR_CUDA;
    if (detail) *detail = word;
    if (word == 0) return SQ_OK;
    if (cudaMemsetAsync(workspace, 0, sizeof(word), st) != cudaSuccess) return SQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SQ_ERR_CUDA;
    return SQ_ERR_TIMEOUT;
}

sq_status segquant_set_quantize_tuning(int fused_table_mode)
{
    if (fused_table_mode < 0 || fused_table_mode > 2) return SQ_ERR_UNSUPPORTED;
    set_quantize_table_mode(fused_table_mode);
    return SQ_OK;
}

sq_status segquant_set_tuning(int tile_n, int stages, int cta_group, int segment_mode)
{
    set_gemm_tuning(tile_n, stages, cta_group, segment_mode);
    return SQ_OK;
}

const char *segquant_last_cuda_error(void)
{
    return cudaGetErrorString(cudaError_t(g_last_cuda_error.load(std::memory_order_relaxed)));
}

uint64_t segquant_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *segquant_status_string(sq_status s)
{
    switch (s) {
        case SQ_OK: return "ok";
        case SQ_ERR_NULL: return "null pointer";
        case SQ_ERR_SHAPE: return "bad shape";
        case SQ_ERR_SEGTABLE: return "bad segment table";
        case SQ_ERR_ALIGN: return "alignment";
        case SQ_ERR_UNSUPPORTED: return "unsupported";
        case SQ_ERR_CUDA: return "cuda error";
        case SQ_ERR_TIMEOUT: return "device wait timed out";
        case SQ_ERR_WORKSPACE: return "workspace missing or too small";
    }
    return "unknown";
}

}  // extern "C"
