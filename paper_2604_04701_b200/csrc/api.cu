// C-ABI host layer of libmuxq: argument checks, workspace carving, kernel launches.
// No device memory is allocated here; the only host state that survives a call is the per-device record of
// one-time set-up (host_state.cu).
#include <math.h>
#include <string.h>

#include "../../include/muxq.h"
#include "../../include/muxq_measure.h"
#include "kernels.h"

using namespace muxq;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool params_ok(const muxq_params *p) {
    return p && p->exp_factor >= 1 && p->exp_factor <= 3 && p->act_bits >= 2 && p->act_bits <= 8 &&
           p->w_bits >= 2 && p->w_bits <= 8 && (p->gran == MUXQ_PER_TENSOR || p->gran == MUXQ_PER_VECTOR) &&
           (p->aux_scale == MUXQ_AUX_SHARED || p->aux_scale == MUXQ_AUX_OWN) && p->max_outliers >= 1 &&
           p->max_outliers <= kMaxOutlierCap && isfinite(p->threshold) && p->threshold >= 0.0f;
}
inline int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

// Small workspace (detect / quantize): ctrl | colmax_bits[cols] | colmul[cols] | grpflag[cols/8] | oidx[64]
struct SmallWs {
    size_t ctrl, colmax, colmul, grpflag, oidx, total;
};
SmallWs small_ws(int cols) {
    SmallWs w;
    w.ctrl = 0;
    w.colmax = sizeof(Ctrl);
    w.colmul = align_up(w.colmax + (size_t)cols * 4, 256);
    w.grpflag = align_up(w.colmul + (size_t)cols * 4, 256);
    w.oidx = align_up(w.grpflag + (size_t)(cols + 7) / 8, 256);
    w.total = align_up(w.oidx + (size_t)kMaxOutlierCap * 4, 256);
    return w;
}

// muxq_linear workspace: the small block, then per-token scales, Body_q, Aux_q, W_aux.
struct LinearWs {
    SmallWs s;
    size_t colmax_rep, sx_rows, sa_rows, body_q, aux_q, w_aux, t1, t2, total;
    int ld_q, aux_cols;
};
LinearWs linear_ws(int M, int K, int N, const muxq_params *p) {
    LinearWs w;
    w.s = small_ws(K);
    w.aux_cols = muxq_aux_cols(p);
    w.ld_q = K;
    // The replicated abs-max accumulators of the fused kernel sit right behind ctrl, in a region of fixed
    // size: the fused kernel finds it zero and leaves it zero, for every shape that shares the workspace.
    // Everything a call overwrites with other values follows behind it.
    w.colmax_rep = sizeof(Ctrl);
    const size_t shift = align_up(w.colmax_rep + kPrepRepRegionBytes, 256) - w.s.colmax;
    w.s.colmax += shift; w.s.colmul += shift; w.s.grpflag += shift; w.s.oidx += shift; w.s.total += shift;
    w.sx_rows = w.s.total;
    w.sa_rows = align_up(w.sx_rows + (size_t)M * 4, 256);
    w.body_q = align_up(w.sa_rows + (size_t)M * 4, 1024);
    w.aux_q = align_up(w.body_q + (size_t)M * w.ld_q, 1024);
    w.w_aux = align_up(w.aux_q + (size_t)M * w.aux_cols, 1024);
    w.total = align_up(w.w_aux + (size_t)N * w.aux_cols, 1024);
    // own-scale reading: the two dequantized products, fp32 [M, N] each
    w.t1 = w.t2 = 0;
    if (p->aux_scale == MUXQ_AUX_OWN) {
        w.t1 = w.total;
        w.t2 = align_up(w.t1 + (size_t)M * N * 4, 1024);
        w.total = align_up(w.t2 + (size_t)M * N * 4, 1024);
    }
    return w;
}

inline size_t out_elem_bytes(int out_kind) { return out_kind == MUXQ_OUT_F16 ? 2 : 4; }

int cuda_rc(cudaError_t e) { return e == cudaSuccess ? MUXQ_OK : MUXQ_ERR_CUDA; }

}  // namespace

extern "C" {

void muxq_default_params(muxq_params *p) {
    if (!p) return;
    p->threshold = 6.0f;
    p->exp_factor = 2;
    p->act_bits = 8;
    p->w_bits = 8;
    p->gran = MUXQ_PER_TENSOR;
    p->aux_scale = MUXQ_AUX_SHARED;
    p->max_outliers = 64;
}

int muxq_aux_cols(const muxq_params *p) {
    if (!params_ok(p)) return 0;
    const int c = (1 << p->exp_factor) - 1;
    return (int)align_up((size_t)c * p->max_outliers, 128);
}

size_t muxq_small_workspace_bytes(int cols) { return cols > 0 ? small_ws(cols).total : 0; }

size_t muxq_workspace_bytes(int M, int K, int N, const muxq_params *p) {
    if (M <= 0 || K <= 0 || N <= 0 || !params_ok(p)) return 0;
    return linear_ws(M, K, N, p).total;
}

size_t muxq_host_workspace_bytes(int M, int K, int N, const muxq_params *p, int out_kind) {
    const size_t base = muxq_workspace_bytes(M, K, N, p);
    if (!base || out_kind < 0 || out_kind > 2) return 0;
    return base + align_up((size_t)M * K * 2, 1024) + align_up((size_t)M * N * out_elem_bytes(out_kind), 1024);
}

int muxq_workspace_init(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace || workspace_bytes < sizeof(Ctrl)) return MUXQ_ERR_INVALID_ARG;
    const size_t n = sizeof(Ctrl) + kPrepRepRegionBytes;
    return cuda_rc(cudaMemsetAsync(workspace, 0, workspace_bytes < n ? workspace_bytes : n,
                                   static_cast<cudaStream_t>(stream)));
}

int muxq_workspace_view(int M, int K, int N, const muxq_params *p, muxq_ws_view *v) {
    if (!v || M <= 0 || K <= 0 || N <= 0 || !params_ok(p)) return MUXQ_ERR_INVALID_ARG;
    const LinearWs w = linear_ws(M, K, N, p);
    v->col_absmax = w.s.colmax;
    v->outlier_idx = w.s.oidx;
    v->n_outliers = offsetof(Ctrl, n_outliers);
    v->s_x = p->gran == MUXQ_PER_VECTOR ? w.sx_rows : offsetof(Ctrl, s_x);
    v->s_a = p->gran == MUXQ_PER_VECTOR ? w.sa_rows : offsetof(Ctrl, s_a);
    v->body_q = w.body_q;
    v->aux_q = w.aux_q;
    v->w_aux = w.w_aux;
    v->ld_body_q = w.ld_q;
    v->aux_cols = w.aux_cols;
    return MUXQ_OK;
}

int muxq_detect_outliers(const void *X, int M, int K, int ldx, float threshold, float *col_absmax,
                         int32_t *outlier_idx, int32_t *n_outliers, int cap, void *workspace,
                         size_t workspace_bytes, void *stream) {
    if (!X || !col_absmax || !outlier_idx || !n_outliers || !workspace || M <= 0 || K <= 0 || ldx < K ||
        cap < 1 || !(threshold >= 0.0f))
        return MUXQ_ERR_INVALID_ARG;
    if (K % 8 || ldx % 8 || !aligned16(X) || !aligned16(col_absmax) || !aligned16(workspace))
        return MUXQ_ERR_UNSUPPORTED;
    if (workspace_bytes < sizeof(Ctrl)) return MUXQ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(workspace, 0, sizeof(Ctrl), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(col_absmax, 0, (size_t)K * 4, s);
    if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    DetectArgs a{};
    a.X = static_cast<const __half *>(X);
    a.M = M; a.K = K; a.ldx = ldx;
    a.tau = threshold; a.exp_factor = 0; a.qmax = 127; a.cap = cap;
    a.colmax_bits = reinterpret_cast<uint32_t *>(col_absmax);
    a.ctrl = static_cast<Ctrl *>(workspace);
    a.outlier_idx = outlier_idx;
    a.n_outliers = n_outliers;
    return cuda_rc(launch_detect(a, s));
}

int muxq_build_aux(const void *X, int M, int K, int ldx, const int32_t *outlier_idx, const int32_t *n_outliers,
                   int cap, int exp_factor, float *Aux, int ld_aux, float *Body, int ld_body, void *stream) {
    if (!X || !outlier_idx || !n_outliers || !Aux || M <= 0 || K <= 0 || ldx < K || cap < 1 || ld_aux < cap ||
        exp_factor < 1 || exp_factor > 3 || (Body && ld_body < K))
        return MUXQ_ERR_INVALID_ARG;
    BuildAuxArgs a{static_cast<const __half *>(X), M, K, ldx, outlier_idx, n_outliers, cap, exp_factor,
                   Aux, ld_aux, Body, ld_body};
    return cuda_rc(launch_build_aux(a, static_cast<cudaStream_t>(stream)));
}

int muxq_quantize(const void *A, int rows, int cols, int ld, const muxq_params *p, int is_weight,
                  const float *col_absmax, const int32_t *outlier_idx, const int32_t *n_outliers, int8_t *A_q,
                  int ld_q, int8_t *Aux_q, int ld_aux, float *scales, void *workspace, size_t workspace_bytes,
                  void *stream) {
    if (!A || !A_q || !scales || !workspace || rows <= 0 || cols <= 0 || ld < cols || !params_ok(p))
        return MUXQ_ERR_INVALID_ARG;
    if (cols % 8 || ld % 8 || !aligned16(A) || !aligned16(workspace) || !aligned16(A_q))
        return MUXQ_ERR_UNSUPPORTED;
    if (workspace_bytes < muxq_small_workspace_bytes(cols)) return MUXQ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const SmallWs w = small_ws(cols);

    if (is_weight) {
        // A = W [K=rows, N=cols]; abs-max per output channel n through the same reduction as K1
        if (ld_q < rows) return MUXQ_ERR_INVALID_ARG;
        cudaError_t e = cudaMemsetAsync(ws, 0, w.colmax + (size_t)cols * 4, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
        DetectArgs d{};
        d.X = static_cast<const __half *>(A);
        d.M = rows; d.K = cols; d.ldx = ld;
        d.tau = INFINITY; d.exp_factor = 0; d.qmax = qmax_of(p->w_bits); d.cap = 0;
        d.colmax_bits = reinterpret_cast<uint32_t *>(ws + w.colmax);
        d.ctrl = reinterpret_cast<Ctrl *>(ws);
        d.outlier_idx = reinterpret_cast<int32_t *>(ws + w.oidx);
        e = launch_detect(d, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
        QuantWeightArgs q{};
        q.W = static_cast<const __half *>(A);
        q.K = rows; q.N = cols; q.ldw = ld;
        q.qmax = qmax_of(p->w_bits);
        q.per_channel = p->gran == MUXQ_PER_VECTOR;
        q.colmax_bits = d.colmax_bits;
        q.s_tensor = &d.ctrl->s_x;
        q.s_w = scales;
        q.w_q = A_q; q.ld_q = ld_q;
        return cuda_rc(launch_quant_weight(q, s));
    }

    // activations: A = X [M=rows, K=cols]
    if (!col_absmax || (outlier_idx == nullptr) != (n_outliers == nullptr) || ld_q < cols)
        return MUXQ_ERR_INVALID_ARG;
    if (p->aux_scale != MUXQ_AUX_SHARED) return MUXQ_ERR_UNSUPPORTED;
    const int aux_cols = muxq_aux_cols(p);
    if (Aux_q && (ld_aux < aux_cols || ld_aux % 4 || (reinterpret_cast<uintptr_t>(Aux_q) & 3u)))
        return MUXQ_ERR_INVALID_ARG;
    if (ld_q % 8) return MUXQ_ERR_UNSUPPORTED;
    cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(Ctrl), s);
    if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    DetectArgs d{};
    d.X = static_cast<const __half *>(A);
    d.M = rows; d.K = cols; d.ldx = ld;
    d.tau = outlier_idx ? p->threshold : INFINITY;
    d.exp_factor = p->exp_factor; d.qmax = qmax_of(p->act_bits); d.cap = p->max_outliers;
    d.colmax_bits = reinterpret_cast<uint32_t *>(const_cast<float *>(col_absmax));  // read-only in the tail
    d.ctrl = reinterpret_cast<Ctrl *>(ws);
    d.outlier_idx = reinterpret_cast<int32_t *>(ws + w.oidx);
    d.colmul = reinterpret_cast<float *>(ws + w.colmul);
    d.grpflag = ws + w.grpflag;
    e = launch_detect_finalize(d, s);
    if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    QuantActArgs q{};
    q.X = d.X; q.M = rows; q.K = cols; q.ldx = ld;
    q.exp_factor = p->exp_factor; q.qmax = d.qmax; q.cap = p->max_outliers;
    q.per_token = p->gran == MUXQ_PER_VECTOR;
    q.outlier_idx = d.outlier_idx;
    q.n_outliers = &d.ctrl->n_outliers;
    q.colmul = d.colmul; q.grpflag = d.grpflag;
    q.s_x_tensor = &d.ctrl->s_x;
    q.inv_s_x_tensor = &d.ctrl->inv_s_x;
    q.s_x_rows = scales;
    q.body_q = A_q; q.ld_q = ld_q;
    q.aux_q = Aux_q; q.ld_aux = ld_aux; q.aux_cols = aux_cols;
    e = launch_quant_act(q, s);
    if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    if (!q.per_token) e = cudaMemcpyAsync(scales, &d.ctrl->s_x, 4, cudaMemcpyDeviceToDevice, s);
    return cuda_rc(e);
}

int muxq_gemm(const int8_t *Body_q, int ld_a, const int8_t *Aux_q, int ld_aux, const int8_t *W_q, int ldw,
              const int8_t *W_aux, int ld_waux, const int32_t *n_outliers, int M, int K, int N,
              const muxq_params *p, const float *s_x, const float *s_w, void *Y, int ldy, int out_kind,
              int32_t *dev_status, void *stream) {
    if (!Body_q || !W_q || !Y || M <= 0 || K <= 0 || N <= 0 || ld_a < K || ldw < K || ldy < N || !params_ok(p) ||
        out_kind < 0 || out_kind > 2 || (out_kind != MUXQ_OUT_ACC_I32 && (!s_x || !s_w)))
        return MUXQ_ERR_INVALID_ARG;
    const bool has_aux = Aux_q && W_aux && n_outliers;
    const int aux_cols = muxq_aux_cols(p);
    if (has_aux && (ld_aux < aux_cols || ld_waux < aux_cols)) return MUXQ_ERR_INVALID_ARG;
    const int yal = out_kind == MUXQ_OUT_F16 ? 8 : 4;
    if (K % 16 || ld_a % 16 || ldw % 16 || N % 8 || ldy % yal || !aligned16(Body_q) || !aligned16(W_q) ||
        !aligned16(Y) || (has_aux && (ld_aux % 16 || ld_waux % 16 || !aligned16(Aux_q) || !aligned16(W_aux))) ||
        (p->gran == MUXQ_PER_VECTOR && s_w && !aligned16(s_w)))
        return MUXQ_ERR_UNSUPPORTED;
    if (p->aux_scale != MUXQ_AUX_SHARED) return MUXQ_ERR_UNSUPPORTED;
    GemmArgs g{};
    g.body_q = Body_q; g.ld_a = ld_a;
    g.aux_q = has_aux ? Aux_q : nullptr; g.ld_aux = ld_aux;
    g.w_q = W_q; g.ldw = ldw;
    g.w_aux = has_aux ? W_aux : nullptr; g.ld_waux = ld_waux;
    g.n_outliers = has_aux ? n_outliers : nullptr;
    g.M = M; g.K = K; g.N = N;
    g.c = (1 << p->exp_factor) - 1; g.cap = p->max_outliers; g.aux_cols = aux_cols;
    g.s_x = s_x; g.s_x_per_row = p->gran == MUXQ_PER_VECTOR;
    g.s_w = s_w; g.s_w_per_col = p->gran == MUXQ_PER_VECTOR;
    g.Y = Y; g.ldy = ldy; g.out_kind = out_kind;
    g.dev_status = dev_status;
    return cuda_rc(launch_gemm(g, static_cast<cudaStream_t>(stream)));
}

static int linear_impl(const void *X, int M, int K, int ldx, const int8_t *W_q, int ldw, const float *s_w,
                       const float *bias, int N, const muxq_params *p, void *Y, int ldy, int out_kind, void *workspace, size_t workspace_bytes,
                       int32_t *dev_status, void *stream, void *const *events) {
    if (!X || !W_q || !s_w || !Y || !workspace || !dev_status || M <= 0 || K <= 0 || N <= 0 || ldx < K ||
        ldw < K || ldy < N || !params_ok(p) || out_kind < 0 || out_kind > 2)
        return MUXQ_ERR_INVALID_ARG;
    const int yal = out_kind == MUXQ_OUT_F16 ? 8 : 4;
    if (K % 16 || ldx % 8 || ldw % 16 || N % 8 || ldy % yal || !aligned16(X) || !aligned16(W_q) ||
        !aligned16(Y) || !aligned16(workspace) || (p->gran == MUXQ_PER_VECTOR && !aligned16(s_w)))
        return MUXQ_ERR_UNSUPPORTED;
    const bool aux_own = p->aux_scale == MUXQ_AUX_OWN;
    if (aux_own && out_kind == MUXQ_OUT_ACC_I32) return MUXQ_ERR_UNSUPPORTED;  // there is no common accumulator
    if (bias && out_kind == MUXQ_OUT_ACC_I32) return MUXQ_ERR_INVALID_ARG;     // the bias belongs to the dequantized output
    if (bias && (aux_own || !aligned16(bias))) return MUXQ_ERR_UNSUPPORTED;
    const LinearWs w = linear_ws(M, K, N, p);
    if (workspace_bytes < w.total) return MUXQ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);

    const bool per_vec = p->gran == MUXQ_PER_VECTOR;
    // (the own-scale reading runs as separate products through the GEMM kernels for every M)
    const bool decode = M <= 16 && !aux_own;
    const bool fused = prep_supported(M, K);
    if (aux_own && !fused) return MUXQ_ERR_UNSUPPORTED;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(ws);
    // inside a stream capture the records become event-record nodes that every replay re-records
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (events) cudaStreamIsCapturing(s, &cap);
    const unsigned ev_flags = cap == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault;
    auto mark = [&](int i) {
        if (events && events[i]) cudaEventRecordWithFlags(static_cast<cudaEvent_t>(events[i]), s, ev_flags);
    };
    mark(0);
    if (decode && decode_fused_supported(M, K)) {
        // M <= 16: one launch does the whole layer and needs no cleared scratch; it leaves colmax, O, r
        // and the scale(s) in the workspace for inspection
        DecodeFusedArgs k{};
        k.X = static_cast<const __half *>(X);
        k.M = M; k.K = K; k.ldx = ldx;
        k.w_q = W_q; k.ldw = ldw; k.N = N;
        k.s_w = s_w; k.per_vec = per_vec;
        k.bias = bias;
        k.tau = p->threshold; k.exp_factor = p->exp_factor; k.qmax = qmax_of(p->act_bits);
        k.cap = p->max_outliers; k.c = (1 << p->exp_factor) - 1;
        k.Y = Y; k.ldy = ldy; k.out_kind = out_kind;
        k.colmax = reinterpret_cast<float *>(ws + w.s.colmax);
        k.outlier_idx = reinterpret_cast<int32_t *>(ws + w.s.oidx);
        k.ctrl = ctrl;
        k.s_x_rows = reinterpret_cast<float *>(ws + w.sx_rows);
        k.dev_status = dev_status;
        mark(1);
        mark(2);
        const cudaError_t ed = launch_decode_fused(k, s);
        mark(3);
        return cuda_rc(ed);
    }
    // The fused kernel keeps its counters and accumulators zero between calls (muxq_workspace_init zeroed
    // them once); the separate kernels take a cleared control block and abs-max array per call.
    cudaError_t e = cudaSuccess;
    if (!fused) {
        e = cudaMemsetAsync(ws, 0, sizeof(Ctrl), s);
        if (e == cudaSuccess) e = cudaMemsetAsync(ws + w.s.colmax, 0, (size_t)K * 4, s);
    }
    if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    mark(1);

    int32_t *oidx = reinterpret_cast<int32_t *>(ws + w.s.oidx);
    float *s_x_rows = reinterpret_cast<float *>(ws + w.sx_rows);
    int8_t *body_q = reinterpret_cast<int8_t *>(ws + w.body_q);
    int8_t *aux_q = decode ? nullptr : reinterpret_cast<int8_t *>(ws + w.aux_q);
    int8_t *w_aux = decode ? nullptr : reinterpret_cast<int8_t *>(ws + w.w_aux);
    if (fused) {
        PrepArgs f{};
        f.X = static_cast<const __half *>(X);
        f.M = M; f.K = K; f.ldx = ldx;
        f.tau = p->threshold; f.exp_factor = p->exp_factor; f.qmax = qmax_of(p->act_bits);
        f.cap = p->max_outliers; f.per_token = per_vec;
        f.aux_own = aux_own ? 1 : 0;
        f.s_a_rows = reinterpret_cast<float *>(ws + w.sa_rows);
        f.colmax_rep = reinterpret_cast<uint32_t *>(ws + w.colmax_rep);
        f.colmax_bits = reinterpret_cast<uint32_t *>(ws + w.s.colmax);
        f.ctrl = ctrl;
        f.outlier_idx = oidx;
        f.s_x_rows = s_x_rows;
        f.body_q = body_q; f.ld_q = w.ld_q;
        f.aux_q = aux_q; f.ld_aux = w.aux_cols; f.aux_cols = w.aux_cols;
        if (!decode) { f.w_q = W_q; f.ldw = ldw; f.N = N; f.w_aux = w_aux; f.ld_waux = w.aux_cols; }
        f.dev_status = dev_status;
        e = launch_prep(f, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    } else {
        DetectArgs d{};
        d.X = static_cast<const __half *>(X);
        d.M = M; d.K = K; d.ldx = ldx;
        d.tau = p->threshold; d.exp_factor = p->exp_factor; d.qmax = qmax_of(p->act_bits); d.cap = p->max_outliers;
        d.colmax_bits = reinterpret_cast<uint32_t *>(ws + w.s.colmax);
        d.ctrl = ctrl;
        d.outlier_idx = oidx;
        d.colmul = reinterpret_cast<float *>(ws + w.s.colmul);
        d.grpflag = ws + w.s.grpflag;
        d.dev_status = dev_status;
        e = launch_detect(d, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
        QuantActArgs q{};
        q.X = d.X; q.M = M; q.K = K; q.ldx = ldx;
        q.exp_factor = p->exp_factor; q.qmax = d.qmax; q.cap = p->max_outliers; q.per_token = per_vec;
        q.outlier_idx = oidx;
        q.n_outliers = &ctrl->n_outliers;
        q.colmul = d.colmul; q.grpflag = d.grpflag;
        q.s_x_tensor = &ctrl->s_x;
        q.inv_s_x_tensor = &ctrl->inv_s_x;
        q.s_x_rows = s_x_rows;
        q.body_q = body_q; q.ld_q = w.ld_q;
        if (!decode) {
            q.aux_q = aux_q; q.ld_aux = w.aux_cols; q.aux_cols = w.aux_cols;
            q.w_q = W_q; q.ldw = ldw; q.N = N;
            q.w_aux = w_aux; q.ld_waux = w.aux_cols;
        }
        e = launch_quant_act(q, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
    }
    mark(2);

    const float *s_x = per_vec ? s_x_rows : &ctrl->s_x;
    const int c = (1 << p->exp_factor) - 1;
    if (decode) {
        DecodeArgs k{};
        k.body_q = body_q; k.ld_a = w.ld_q;
        k.w_q = W_q; k.ldw = ldw;
        k.outlier_idx = oidx; k.n_outliers = &ctrl->n_outliers;
        k.M = M; k.K = K; k.N = N; k.c = c; k.cap = p->max_outliers;
        k.s_x = s_x; k.s_x_per_row = per_vec;
        k.s_w = s_w; k.s_w_per_col = per_vec;
        k.bias = bias;
        k.Y = Y; k.ldy = ldy; k.out_kind = out_kind;
        e = launch_decode(k, s);
        mark(3);
        return cuda_rc(e);
    }
    if (aux_own) {
        // Y = (s_X s_W) Body_q.W_q + c (s_A s_W) Aux_q.W_aux: two dequantized products, then the sum
        float *t1 = reinterpret_cast<float *>(ws + w.t1), *t2 = reinterpret_cast<float *>(ws + w.t2);
        GemmArgs g{};
        g.body_q = body_q; g.ld_a = w.ld_q;
        g.w_q = W_q; g.ldw = ldw;
        g.M = M; g.K = K; g.N = N; g.c = c; g.cap = p->max_outliers; g.aux_cols = w.aux_cols;
        g.s_x = s_x; g.s_x_per_row = per_vec;
        g.s_w = s_w; g.s_w_per_col = per_vec;
        g.Y = t1; g.ldy = N; g.out_kind = MUXQ_OUT_F32;
        g.dev_status = dev_status;
        e = launch_gemm(g, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
        g.body_q = aux_q; g.ld_a = w.aux_cols;  // zero beyond the r used columns
        g.w_q = w_aux; g.ldw = w.aux_cols;
        g.K = w.aux_cols;
        g.s_x = per_vec ? reinterpret_cast<const float *>(ws + w.sa_rows) : &ctrl->s_a;
        g.Y = t2;
        e = launch_gemm(g, s);
        if (e != cudaSuccess) return MUXQ_ERR_CUDA;
        CombineArgs cb{t1, t2, M, N, c, Y, ldy, out_kind == MUXQ_OUT_F16 ? 1 : 0};
        e = launch_combine(cb, s);
        mark(3);
        return cuda_rc(e);
    }
    GemmArgs g{};
    g.body_q = body_q; g.ld_a = w.ld_q;
    g.aux_q = aux_q; g.ld_aux = w.aux_cols;
    g.w_q = W_q; g.ldw = ldw;
    g.w_aux = w_aux; g.ld_waux = w.aux_cols;
    g.n_outliers = &ctrl->n_outliers;
    g.M = M; g.K = K; g.N = N; g.c = c; g.cap = p->max_outliers; g.aux_cols = w.aux_cols;
    g.s_x = s_x; g.s_x_per_row = per_vec;
    g.s_w = s_w; g.s_w_per_col = per_vec;
    g.bias = bias;
    g.Y = Y; g.ldy = ldy; g.out_kind = out_kind;
    g.dev_status = dev_status;
    g.w_stable = 1;  // the kernel before this one in the stream is the preparation of X, which does not write W_q
    e = launch_gemm(g, s);
    mark(3);
    return cuda_rc(e);
}

int muxq_linear(const void *X, int M, int K, int ldx, const int8_t *W_q, int ldw, const float *s_w, int N,
                const muxq_params *p, void *Y, int ldy, int out_kind, void *workspace, size_t workspace_bytes,
                int32_t *dev_status, void *stream) {
    return linear_impl(X, M, K, ldx, W_q, ldw, s_w, nullptr, N, p, Y, ldy, out_kind, workspace, workspace_bytes,
                       dev_status, stream, nullptr);
}

int muxq_linear_bias(const void *X, int M, int K, int ldx, const int8_t *W_q, int ldw, const float *s_w,
                     const float *bias, int N, const muxq_params *p, void *Y, int ldy, int out_kind, void *workspace,
                     size_t workspace_bytes, int32_t *dev_status, void *stream) {
    return linear_impl(X, M, K, ldx, W_q, ldw, s_w, bias, N, p, Y, ldy, out_kind, workspace, workspace_bytes,
                       dev_status, stream, nullptr);
}

int muxq_linear_events(const void *X, int M, int K, int ldx, const int8_t *W_q, int ldw, const float *s_w, int N,
                       const muxq_params *p, void *Y, int ldy, int out_kind, void *workspace,
                       size_t workspace_bytes, int32_t *dev_status, void *stream, void *const *events) {
    if (!events) return MUXQ_ERR_INVALID_ARG;
    return linear_impl(X, M, K, ldx, W_q, ldw, s_w, nullptr, N, p, Y, ldy, out_kind, workspace, workspace_bytes,
                       dev_status, stream, events);
}

int muxq_linear_host(const void *X_host, int M, int K, const int8_t *W_q, int ldw, const float *s_w, int N,
                     const muxq_params *p, void *Y_host, int out_kind, void *workspace, size_t workspace_bytes,
                     int32_t *dev_status, void *stream) {
    if (!X_host || !Y_host || !workspace) return MUXQ_ERR_INVALID_ARG;
    const size_t need = muxq_host_workspace_bytes(M, K, N, p, out_kind);
    if (!need) return MUXQ_ERR_INVALID_ARG;
    if (workspace_bytes < need) return MUXQ_ERR_WORKSPACE;
    const size_t base = muxq_workspace_bytes(M, K, N, p);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *x_dev = ws + base;
    uint8_t *y_dev = x_dev + align_up((size_t)M * K * 2, 1024);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(x_dev, X_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return MUXQ_ERR_CUDA;
    const int rc = muxq_linear(x_dev, M, K, K, W_q, ldw, s_w, N, p, y_dev, N, out_kind, ws, base, dev_status, stream);
    if (rc != MUXQ_OK) return rc;
    return cuda_rc(cudaMemcpyAsync(Y_host, y_dev, (size_t)M * N * out_elem_bytes(out_kind), cudaMemcpyDeviceToHost, s));
}

int muxq_int8_mma_peak(int mma_n, int iters, int ctas, unsigned long long *cycles_per_cta, int32_t *dev_status,
                       void *stream) {
    if ((mma_n != 128 && mma_n != 256 && mma_n != 16 && mma_n != 64) || iters < 1 || iters > (1 << 20) || ctas < 1 || !cycles_per_cta)
        return MUXQ_ERR_INVALID_ARG;
    return cuda_rc(launch_mma_peak(mma_n, iters, cycles_per_cta, dev_status, ctas, static_cast<cudaStream_t>(stream)));
}

// ---------------------------------------------------------------- a list of decode-shaped layers in one launch
namespace {
constexpr uint32_t kPlanMagic = 0x4d555851u;
struct PlanHeader {           // first 128 bytes of a plan (host and device copy alike)
    uint32_t magic;
    int32_t n_layers, M, kmax, grid, out_kind;
    muxq_params params;
    uint64_t sync_off, scratch_off, device_bytes;  // layout of the device copy behind the two tables
    int32_t slots, lgroups, xregion;               // shared-memory geometry (chain_geometry)
    uint32_t reserved[5];
};
static_assert(sizeof(PlanHeader) <= 128, "plan header");
constexpr size_t kPlanTableOffset = 128;
// behind the header: the layer table, then one word per layer (its place in shared memory), then counters and scratch
size_t plan_place_offset(int n_layers) { return kPlanTableOffset + (size_t)n_layers * sizeof(ChainLayer); }
size_t plan_sync_offset(int n_layers) { return align_up(plan_place_offset(n_layers) + (size_t)n_layers * 4, 128); }
}  // namespace

size_t muxq_chain_plan_bytes(int n_layers) {
    if (n_layers < 1 || n_layers > kChainMaxLayers) return 0;
    return plan_sync_offset(n_layers);
}

size_t muxq_chain_device_bytes(const muxq_layer *layers, int n_layers, int M) {
    if (!layers || n_layers < 1 || n_layers > kChainMaxLayers || M < 1 || M > 16) return 0;
    size_t scratch = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (layers[l].K <= 0 || layers[l].K % 64) return 0;
        ChainLayer one{};
        one.K = layers[l].K;
        scratch += chain_scratch_bytes(&one, 1, M);
    }
    return plan_sync_offset(n_layers) + chain_sync_bytes(n_layers) + scratch;
}

int muxq_chain_build(const muxq_layer *layers, int n_layers, int M, const muxq_params *p, int out_kind,
                     void *plan_host, size_t plan_host_bytes, void *plan_dev, size_t plan_dev_bytes, void *stream) {
    if (!layers || !plan_host || !plan_dev || n_layers < 1 || M < 1 || !params_ok(p) || out_kind < 0 || out_kind > 2)
        return MUXQ_ERR_INVALID_ARG;
    if (n_layers > kChainMaxLayers || M > 16 || p->aux_scale != MUXQ_AUX_SHARED) return MUXQ_ERR_UNSUPPORTED;
    if (plan_host_bytes < muxq_chain_plan_bytes(n_layers)) return MUXQ_ERR_WORKSPACE;
    if (!aligned16(plan_dev)) return MUXQ_ERR_UNSUPPORTED;
    const int grid = num_sms();
    if (grid < 1) return MUXQ_ERR_CUDA;
    PlanHeader *h = static_cast<PlanHeader *>(plan_host);
    ChainLayer *tab = reinterpret_cast<ChainLayer *>(static_cast<uint8_t *>(plan_host) + kPlanTableOffset);
    memset(h, 0, sizeof(PlanHeader));
    const int yal = out_kind == MUXQ_OUT_F16 ? 8 : 4;
    for (int l = 0; l < n_layers; ++l) {
        const muxq_layer &in = layers[l];
        if (!in.X_f16 || !in.W_q || !in.s_w || !in.Y || in.K <= 0 || in.N <= 0 || in.ldx < in.K || in.ldw < in.K ||
            in.ldy < in.N || (in.flags & ~MUXQ_LAYER_WAIT_PREV) || (l == 0 && in.flags) ||
            (in.bias && out_kind == MUXQ_OUT_ACC_I32))
            return MUXQ_ERR_INVALID_ARG;
        if (!chain_layer_supported(M, in.K, in.N) || in.ldx % 8 || in.ldw % 16 || in.ldy % yal || !aligned16(in.X_f16) ||
            !aligned16(in.W_q) || !aligned16(in.Y) || (p->gran == MUXQ_PER_VECTOR && !aligned16(in.s_w)))
            return MUXQ_ERR_UNSUPPORTED;
        ChainLayer &o = tab[l];
        o.X = static_cast<const __half *>(in.X_f16);
        o.w_q = in.W_q;
        o.s_w = in.s_w;
        o.Y = in.Y;
        o.bias = out_kind == MUXQ_OUT_ACC_I32 ? nullptr : in.bias;
        o.reserved = 0;
        o.ldx = in.ldx; o.ldw = in.ldw; o.ldy = in.ldy; o.K = in.K; o.N = in.N;
        o.flags = (in.flags & MUXQ_LAYER_WAIT_PREV) ? kChainWaitPrev : 0;
    }
    const int kmax = chain_plan(tab, n_layers, grid, chain_slot_bytes(M));
    if (kmax < 0) return MUXQ_ERR_UNSUPPORTED;
    h->sync_off = plan_sync_offset(n_layers);
    h->scratch_off = h->sync_off + chain_sync_bytes(n_layers);
    h->device_bytes = h->scratch_off + chain_scratch_bytes(tab, n_layers, M);
    if (plan_dev_bytes < h->device_bytes) return MUXQ_ERR_WORKSPACE;
    ChainGeometry geo{};
    if (!chain_geometry(tab, n_layers, M, chain_slot_bytes(M), &geo,
                        reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(plan_host) + plan_place_offset(n_layers))))
        return MUXQ_ERR_UNSUPPORTED;
    h->slots = geo.slots; h->lgroups = geo.lgroups; h->xregion = geo.xregion;
    h->magic = kPlanMagic;
    h->n_layers = n_layers; h->M = M; h->kmax = kmax; h->grid = grid; h->out_kind = out_kind;
    h->params = *p;
    // the rows of codes beyond M in the scratch areas are read (as zero) and never written
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(static_cast<uint8_t *>(plan_dev) + h->scratch_off, 0, h->device_bytes - h->scratch_off, s) != cudaSuccess)
        return MUXQ_ERR_CUDA;
    return cuda_rc(cudaMemcpyAsync(plan_dev, plan_host, muxq_chain_plan_bytes(n_layers), cudaMemcpyHostToDevice, s));
}

int muxq_chain_run(const void *plan_host, void *plan_dev, muxq_chain_result *results, int32_t *dev_status,
                   void *stream) {
    if (!plan_host || !plan_dev || !dev_status) return MUXQ_ERR_INVALID_ARG;
    const PlanHeader *h = static_cast<const PlanHeader *>(plan_host);
    if (h->magic != kPlanMagic || h->grid != num_sms()) return MUXQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t *pd = static_cast<uint8_t *>(plan_dev);
    ChainArgs a{};
    a.layers = reinterpret_cast<const ChainLayer *>(pd + kPlanTableOffset);
    a.n_layers = h->n_layers; a.M = h->M; a.kmax = h->kmax; a.grid = h->grid;
    a.tau = h->params.threshold; a.exp_factor = h->params.exp_factor; a.qmax = qmax_of(h->params.act_bits);
    a.cap = h->params.max_outliers; a.c = (1 << h->params.exp_factor) - 1;
    a.per_vec = h->params.gran == MUXQ_PER_VECTOR; a.out_kind = h->out_kind;
    a.results = reinterpret_cast<ChainResult *>(results);
    a.dev_status = dev_status;
    a.spin = test_hooks().spin_limit ? test_hooks().spin_limit : (1u << 22);
    a.extra_arrivals = test_hooks().prep_extra_arrivals;
    a.slot_bytes = chain_slot_bytes(h->M);
    a.sync = pd + h->sync_off;
    a.scratch = pd + h->scratch_off;
    a.slots = h->slots; a.lgroups = h->lgroups; a.xregion = h->xregion;
    a.place = reinterpret_cast<const uint32_t *>(pd + plan_place_offset(h->n_layers));
    // the per-layer counters and maxima start every run at zero
    if (cudaMemsetAsync(a.sync, 0, chain_sync_bytes(h->n_layers), s) != cudaSuccess) return MUXQ_ERR_CUDA;
    return cuda_rc(launch_decode_chain(a, s));
}

int muxq_test_hooks(const muxq_test_hooks_t *h) {
    TestHooks t{};
    if (h) {
        if (h->gemm_skip_k_block < 0) return MUXQ_ERR_INVALID_ARG;
        t.spin_limit = h->spin_limit;
        t.prep_extra_arrivals = h->prep_extra_arrivals;
        t.gemm_skip_kb = h->gemm_skip_k_block;
    }
    set_test_hooks(t);
    return MUXQ_OK;
}

int muxq_read_status(const int32_t *dev_status, void *stream) {
    if (!dev_status) return MUXQ_ERR_INVALID_ARG;
    int32_t h = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&h, dev_status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MUXQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MUXQ_ERR_CUDA;
    return h;
}

const char *muxq_status_string(int st) {
    switch (st) {
        case MUXQ_OK: return "ok";
        case MUXQ_ERR_INVALID_ARG: return "invalid argument";
        case MUXQ_ERR_UNSUPPORTED: return "unsupported shape, alignment or mode";
        case MUXQ_ERR_WORKSPACE: return "workspace too small";
        case MUXQ_ERR_CUDA: return "CUDA runtime error";
        case MUXQ_ERR_CAPACITY: return "more outlier channels than max_outliers";
        case MUXQ_ERR_TIMEOUT: return "bounded device-side wait expired";
        case MUXQ_ERR_STATIC_LIMIT: return "M or K exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

}  // extern "C"
