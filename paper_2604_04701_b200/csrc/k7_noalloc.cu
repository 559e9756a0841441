// muxq_linear_decode_noalloc: the decode-shaped layer (M <= 16 token rows) for callers that cannot
// hand the library a workspace because they cannot allocate device memory at the point of the call:
// code running between the steps of a latency-critical decode loop where cudaMalloc would
// synchronise the whole device, plug-ins loaded into a host process that owns all device memory
// through its own pool, and code that runs after the process has locked its memory budget.
//
// The scratch that muxq_linear takes as its `workspace` argument lives here in a file-scope device
// array of fixed size.  Its device address is looked up once per device with cudaGetSymbolAddress
// (the array's name is only a host-side handle in host code) and passed to the same kernels the
// workspace path launches.  Every call reuses the array, so calls that overlap on the GPU race;
// what has to start at zero is cleared at the head of every call.
#include <math.h>

#include <mutex>

#include "../../include/muxq.h"
#include "kernels.h"

namespace muxq {

namespace {

constexpr int kNoallocMaxM = 16;
constexpr int kNoallocMaxK = 8192;
constexpr int kMaxOutliers = 64;

constexpr size_t align256(size_t v) { return (v + 255) / 256 * 256; }

// ctrl | colmax [K] | colmax replicas [R, K] | outlier_idx [64] | s_x rows [16] | Body_q [16, K]
struct Layout {
    size_t colmax, colmax_rep, oidx, sx_rows, body_q, total;
};
constexpr Layout layout_for(int K) {
    Layout l{};
    l.colmax = sizeof(Ctrl);
    l.colmax_rep = align256(l.colmax + (size_t)K * 4);
    l.oidx = align256(l.colmax_rep + (size_t)kPrepColmaxReplicas * K * 4);
    l.sx_rows = align256(l.oidx + kMaxOutliers * 4);
    l.body_q = align256(l.sx_rows + kNoallocMaxM * 4);
    l.total = align256(l.body_q + (size_t)kNoallocMaxM * K);
    return l;
}
constexpr size_t kScratchBytes = layout_for(kNoallocMaxK).total;
static_assert(kScratchBytes == 426752, "documented size of the built-in scratch");

static __device__ __align__(256) uint8_t g_noalloc_scratch[kScratchBytes];

uint8_t *g_scratch_ptr[kMaxDevices];  // device address of the array on each device, once looked up
std::mutex g_setup_mutex;

// Device address of the scratch array on the current device (set-up on first use per device).
cudaError_t scratch_for_current_device(uint8_t **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = static_cast<uint8_t *>(p);
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace muxq

using namespace muxq;

extern "C" int muxq_linear_decode_noalloc(const void *X, int M, int K, int ldx, const int8_t *W_q, int ldw,
                                          const float *s_w, int N, const muxq_params *p, void *Y, int ldy,
                                          int out_kind, int32_t *dev_status, void *stream) {
    if (!X || !W_q || !s_w || !Y || !dev_status || !p || M <= 0 || K <= 0 || N <= 0 || ldx < K || ldw < K ||
        ldy < N || out_kind < 0 || out_kind > 2 || p->exp_factor < 1 || p->exp_factor > 3 || p->act_bits < 2 ||
        p->act_bits > 8 || p->w_bits < 2 || p->w_bits > 8 || p->max_outliers < 1 || p->max_outliers > kMaxOutliers ||
        (p->gran != MUXQ_PER_TENSOR && p->gran != MUXQ_PER_VECTOR) ||
        (p->aux_scale != MUXQ_AUX_SHARED && p->aux_scale != MUXQ_AUX_OWN) || !(p->threshold >= 0.0f) ||
        !(p->threshold < INFINITY))
        return MUXQ_ERR_INVALID_ARG;
    if (M > kNoallocMaxM || K > kNoallocMaxK) return MUXQ_ERR_STATIC_LIMIT;
    const int yal = out_kind == MUXQ_OUT_F16 ? 8 : 4;
    if (K % 16 || ldx % 8 || ldw % 16 || N % 8 || ldy % yal || !aligned16(X) || !aligned16(W_q) || !aligned16(Y) ||
        p->aux_scale != MUXQ_AUX_SHARED || (p->gran == MUXQ_PER_VECTOR && !aligned16(s_w)))
        return MUXQ_ERR_UNSUPPORTED;

    uint8_t *ws = nullptr;
    if (scratch_for_current_device(&ws) != cudaSuccess) return MUXQ_ERR_CUDA;
    const Layout l = layout_for(K);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the arrival counter and the abs-max accumulators must start at zero; the rest is overwritten
    if (cudaMemsetAsync(ws, 0, l.colmax_rep + (size_t)kPrepColmaxReplicas * K * 4, s) != cudaSuccess)
        return MUXQ_ERR_CUDA;

    const bool per_vec = p->gran == MUXQ_PER_VECTOR;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(ws);
    if (!prep_supported(M, K)) {
        // the widest rows (K beyond what one CTA of the fused kernel covers) take the separate detection and
        // quantization kernels; their two small per-channel arrays use the space of the fused kernel's accumulators
        DetectArgs d{};
        d.X = static_cast<const __half *>(X);
        d.M = M; d.K = K; d.ldx = ldx;
        d.tau = p->threshold; d.exp_factor = p->exp_factor; d.qmax = (1 << (p->act_bits - 1)) - 1;
        d.cap = p->max_outliers;
        d.colmax_bits = reinterpret_cast<uint32_t *>(ws + l.colmax);
        d.ctrl = ctrl;
        d.outlier_idx = reinterpret_cast<int32_t *>(ws + l.oidx);
        d.colmul = reinterpret_cast<float *>(ws + l.colmax_rep);
        d.grpflag = ws + l.colmax_rep + (size_t)K * 4;
        d.dev_status = dev_status;
        if (launch_detect(d, s) != cudaSuccess) return MUXQ_ERR_CUDA;
        QuantActArgs q{};
        q.X = d.X; q.M = M; q.K = K; q.ldx = ldx;
        q.exp_factor = p->exp_factor; q.qmax = d.qmax; q.cap = p->max_outliers; q.per_token = per_vec;
        q.outlier_idx = d.outlier_idx;
        q.n_outliers = &ctrl->n_outliers;
        q.colmul = d.colmul; q.grpflag = d.grpflag;
        q.s_x_tensor = &ctrl->s_x;
        q.inv_s_x_tensor = &ctrl->inv_s_x;
        q.s_x_rows = reinterpret_cast<float *>(ws + l.sx_rows);
        q.body_q = reinterpret_cast<int8_t *>(ws + l.body_q); q.ld_q = K;
        if (launch_quant_act(q, s) != cudaSuccess) return MUXQ_ERR_CUDA;
        DecodeArgs k{};
        k.body_q = q.body_q; k.ld_a = K;
        k.w_q = W_q; k.ldw = ldw;
        k.outlier_idx = d.outlier_idx; k.n_outliers = &ctrl->n_outliers;
        k.M = M; k.K = K; k.N = N; k.c = (1 << p->exp_factor) - 1; k.cap = p->max_outliers;
        k.s_x = per_vec ? q.s_x_rows : &ctrl->s_x; k.s_x_per_row = per_vec;
        k.s_w = s_w; k.s_w_per_col = per_vec;
        k.Y = Y; k.ldy = ldy; k.out_kind = out_kind;
        return launch_decode(k, s) == cudaSuccess ? MUXQ_OK : MUXQ_ERR_CUDA;
    }
    PrepArgs f{};
    f.X = static_cast<const __half *>(X);
    f.M = M; f.K = K; f.ldx = ldx;
    f.tau = p->threshold; f.exp_factor = p->exp_factor; f.qmax = (1 << (p->act_bits - 1)) - 1;
    f.cap = p->max_outliers; f.per_token = per_vec;
    f.colmax_rep = reinterpret_cast<uint32_t *>(ws + l.colmax_rep);
    f.colmax_bits = reinterpret_cast<uint32_t *>(ws + l.colmax);
    f.ctrl = ctrl;
    f.outlier_idx = reinterpret_cast<int32_t *>(ws + l.oidx);
    f.s_x_rows = reinterpret_cast<float *>(ws + l.sx_rows);
    f.body_q = reinterpret_cast<int8_t *>(ws + l.body_q); f.ld_q = K;
    f.dev_status = dev_status;
    if (launch_prep(f, s) != cudaSuccess) return MUXQ_ERR_CUDA;

    DecodeArgs k{};
    k.body_q = f.body_q; k.ld_a = K;
    k.w_q = W_q; k.ldw = ldw;
    k.outlier_idx = f.outlier_idx; k.n_outliers = &ctrl->n_outliers;
    k.M = M; k.K = K; k.N = N; k.c = (1 << p->exp_factor) - 1; k.cap = p->max_outliers;
    k.s_x = per_vec ? f.s_x_rows : &ctrl->s_x; k.s_x_per_row = per_vec;
    k.s_w = s_w; k.s_w_per_col = per_vec;
    k.Y = Y; k.ldy = ldy; k.out_kind = out_kind;
    return launch_decode(k, s) == cudaSuccess ? MUXQ_OK : MUXQ_ERR_CUDA;
}
