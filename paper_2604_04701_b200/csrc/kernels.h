// Internal launch interface between the C-ABI host layer (api.cu) and the kernels.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace muxq {

// ---------------------------------------------------------------- host-side state (host_state.cu)
// The only state the library keeps between calls: results of one-time set-up per device (function attributes
// that were set, occupancy that was queried, the SM count), indexed by the CUDA device ordinal and guarded by
// one mutex, so that a process may drive several GPUs from several threads.
constexpr int kMaxDevices = 64;
template <typename T>
struct PerDevice {
    T v[kMaxDevices];
    bool have[kMaxDevices];
};
int current_device();        // ordinal of the current device, or -1
std::mutex &device_mutex();  // serialises first-use set-up
int num_sms();               // SM count of the current device (0 on error)

// Fault injection for tests, set through muxq_test_hooks (all zero in normal operation): a short poll limit for
// the bounded device-side waits and conditions that make one of them run out without faulting anything.
struct TestHooks {
    uint32_t spin_limit;           // 0 = the kernels' own limits
    uint32_t prep_extra_arrivals;  // the preparation kernel's grid barrier expects this many arrivals that never come
    int32_t gemm_skip_kb;          // 1 + index of a K block whose operand loads the GEMM producer leaves out (0 = none)
};
const TestHooks &test_hooks();
void set_test_hooks(const TestHooks &h);

// Device control block at the start of every workspace.  The stand-alone kernels get it zeroed by a
// memset per call; the fused prep kernel needs `arrived`, `readers` and its replicated abs-max
// accumulators zero on entry and leaves them zero on exit (see k12_prep.cu).
struct Ctrl {
    uint32_t blocks_done;  // K1: CTAs that have merged their partial maxima
    int32_t n_outliers;    // r, true count of outlier channels
    float s_x;             // per-tensor Body scale (Eq. 1)
    float inv_s_x;         // 1 / s_x, correctly rounded (used only to pre-screen the exact division)
    uint32_t arrived;      // fused prep kernel: CTAs that have reached the grid-wide barrier; top bit = a call timed out
    uint32_t readers;      // fused prep kernel: CTAs that have fetched the merged channel maxima
    float s_a;             // per-tensor Aux scale when Aux has its own (Eq. 1 applied to Aux alone)
    uint32_t reserved[57];
};
static_assert(sizeof(Ctrl) == 256, "Ctrl is one 256-byte block");

struct DetectArgs {
    const __half *X;
    int M, K, ldx;
    float tau;
    int exp_factor;   // e
    int qmax;         // 2^(bits-1)-1
    int cap;
    uint32_t *colmax_bits;  // [K] zero-initialised; bit patterns of non-negative floats
    Ctrl *ctrl;             // zero-initialised
    int32_t *outlier_idx;   // [cap] out
    int32_t *n_outliers;    // [1] out (may alias &ctrl->n_outliers)
    float *colmul;          // [K] out or NULL: 2^-e on outlier channels (first cap of them), else 1
    uint8_t *grpflag;       // [K/8] out or NULL: 1 if the 8-column group holds an outlier channel
    float *s_x;             // [1] out or NULL: per-tensor Body scale
    int32_t *dev_status;    // out or NULL: raised to MUXQ_ERR_CAPACITY when r > cap
};
cudaError_t launch_detect(const DetectArgs &a, cudaStream_t s);

// Finalize-only: colmax already complete (used by muxq_quantize on a caller-provided col_absmax).
cudaError_t launch_detect_finalize(const DetectArgs &a, cudaStream_t s);

struct QuantActArgs {
    const __half *X;
    int M, K, ldx;
    int exp_factor, qmax, cap, per_token;
    const int32_t *outlier_idx;  // may be NULL (no outliers)
    const int32_t *n_outliers;   // may be NULL
    const float *colmul;         // [K] or NULL when outlier_idx is NULL
    const uint8_t *grpflag;      // [K/8] or NULL
    const float *s_x_tensor;     // [1] per-tensor scale (device), used when !per_token
    const float *inv_s_x_tensor; // [1] its correctly rounded reciprocal
    float *s_x_rows;             // [M] out when per_token
    int8_t *body_q;  int ld_q;
    int8_t *aux_q;   int ld_aux; int aux_cols;   // aux_q may be NULL
    // W_aux gather fused into the same launch (all NULL/0 to skip)
    const int8_t *w_q; int ldw; int N;
    int8_t *w_aux; int ld_waux;
};
cudaError_t launch_quant_act(const QuantActArgs &a, cudaStream_t s);

// Fused detect + redistribute + quantize (one cooperative launch, X read from HBM once).
constexpr int kMaxOutlierCap = 8192;  // largest max_outliers the entry points accept (every channel of the widest X)
constexpr int kPrepColmaxReplicas = 8;
constexpr int kPrepMaxK = 8192;
// Bytes of replicated accumulators behind Ctrl for the widest supported K.  The region has the same place
// and size for every shape, so "all zero between calls" holds whatever sequence of shapes uses a workspace.
constexpr size_t kPrepRepRegionBytes = (size_t)kPrepColmaxReplicas * kPrepMaxK * 4;
struct PrepArgs {
    const __half *X;
    int M, K, ldx;
    float tau;
    int exp_factor, qmax, cap, per_token;
    int aux_own;             // Aux quantized with its own abs-max scale: columns not repeated, whole block padded with zeros
    float *s_a_rows;         // [M] out when per_token && aux_own
    uint32_t *colmax_rep;    // [kPrepColmaxReplicas, K] accumulators: zero on entry, zeroed again before exit
    uint32_t *colmax_bits;   // [K] out: channel abs-max (bit patterns of non-negative floats)
    Ctrl *ctrl;              // arrived, readers: zero on entry, zero again on exit
    int32_t *outlier_idx;    // [cap] out
    float *s_x_rows;         // [M] out when per_token
    int8_t *body_q;  int ld_q;
    int8_t *aux_q;   int ld_aux; int aux_cols;   // aux_q may be NULL (decode path)
    const int8_t *w_q; int ldw; int N;           // W_aux gather (all NULL/0 to skip)
    int8_t *w_aux; int ld_waux;
    int32_t *dev_status;     // raised (never cleared) on r > cap or when a bounded wait runs out
};
// Own-scale reading: Y = t1 + c * t2 (fp32 in, fp16 or fp32 out); t1, t2 dense [M, N].
struct CombineArgs {
    const float *t1, *t2;
    int M, N, c;
    void *Y; int ldy; int out_f16;
};
cudaError_t launch_combine(const CombineArgs &a, cudaStream_t s);

// False when the shape does not fit the fused kernel (the caller then uses the separate kernels).
bool prep_supported(int M, int K);
cudaError_t launch_prep(const PrepArgs &a, cudaStream_t s);

struct QuantWeightArgs {
    const __half *W;  // [K,N]
    int K, N, ldw;
    int qmax, per_channel;
    const uint32_t *colmax_bits;  // [N] abs-max per output channel (complete)
    const float *s_tensor;        // [1] per-tensor scale (complete)
    float *s_w;                   // [1] or [N] out
    int8_t *w_q; int ld_q;        // [N, ld_q] out
};
cudaError_t launch_quant_weight(const QuantWeightArgs &a, cudaStream_t s);

struct BuildAuxArgs {
    const __half *X; int M, K, ldx;
    const int32_t *outlier_idx; const int32_t *n_outliers; int cap, exp_factor;
    float *aux; int ld_aux; float *body; int ld_body;
};
cudaError_t launch_build_aux(const BuildAuxArgs &a, cudaStream_t s);

struct GemmArgs {
    const int8_t *body_q; int ld_a;
    const int8_t *aux_q;  int ld_aux;
    const int8_t *w_q;    int ldw;
    const int8_t *w_aux;  int ld_waux;
    const int32_t *n_outliers;  // may be NULL
    int M, K, N;
    int c, cap, aux_cols;
    const float *s_x; int s_x_per_row;
    const float *s_w; int s_w_per_col;
    const float *bias;  // [N] fp32 added after the dequantization, or NULL
    void *Y; int ldy; int out_kind;
    int32_t *dev_status;
    int w_stable;  // W_q is not written by the kernel before this one in the stream: its tiles may be fetched early
};
cudaError_t launch_gemm(const GemmArgs &a, cudaStream_t s);
cudaError_t launch_gemm_pair(const GemmArgs &a, int bn, cudaStream_t s);  // two CTAs per 256-row tile

struct DecodeArgs {
    const int8_t *body_q; int ld_a;   // [M, K]
    const int8_t *w_q; int ldw;       // [N, K]
    const int32_t *outlier_idx; const int32_t *n_outliers;
    int M, K, N, c, cap;
    const float *s_x; int s_x_per_row;
    const float *s_w; int s_w_per_col;
    const float *bias;  // [N] fp32 or NULL
    void *Y; int ldy; int out_kind;
};
cudaError_t launch_decode(const DecodeArgs &a, cudaStream_t s);

// Whole layer for M <= 16 in one launch (no scratch needed; the optional outputs are for inspection).
struct DecodeFusedArgs {
    const __half *X; int M, K, ldx;
    const int8_t *w_q; int ldw; int N;
    const float *s_w; int per_vec;      // per-token X scales and per-channel W scales, or one of each
    const float *bias;                  // [N] fp32 added after the dequantization, or NULL
    float tau; int exp_factor, qmax, cap, c;
    void *Y; int ldy; int out_kind;
    float *colmax;                      // [K] out or NULL
    int32_t *outlier_idx;               // [cap] out or NULL
    Ctrl *ctrl;                         // out or NULL: n_outliers, s_x
    float *s_x_rows;                    // [M] out or NULL (per-token scales)
    int32_t *dev_status;                // set to 0, raised to MUXQ_ERR_CAPACITY when r > cap
};
bool decode_fused_supported(int M, int K);
cudaError_t launch_decode_fused(const DecodeFusedArgs &a, cudaStream_t s);

// A list of decode-shaped layers (M <= 16 rows each) in one persistent launch (k4s_decode_stream.cu).
constexpr int kChainMaxLayers = 256;
constexpr int kChainSliceWarps = 7;  // warps per CTA that prepare slices of X for the whole grid
constexpr int kChainWaitPrev = 1;    // ChainLayer::flags bit 0: X of this layer is written by the layer before it
struct ChainLayer {                  // one entry of the device-resident layer table, 80 bytes
    const __half *X;
    const int8_t *w_q;
    const float *s_w;
    void *Y;
    const float *bias;   // [N] fp32 added after the dequantization, or NULL
    uint64_t reserved;
    int ldx, ldw, ldy, K, N, flags;
    // filled by the host (chain_plan):
    uint16_t unit_off;   // unit u of this layer goes to CTA (unit_off + u) mod grid
    uint16_t seg;        // bytes of each W_q row per ring stage (K / seg stages per unit of 8 rows)
    uint16_t slice_off;  // slice s of this layer's X goes to slice warp (slice_off + s) mod (kChainSliceWarps * grid)
    uint16_t nst;        // K / seg
};
static_assert(sizeof(ChainLayer) == 80, "layer table entry");
struct ChainResult {               // per layer, written by CTA 0 (optional)
    int32_t n_outliers;
    int32_t status;                // 0 or MUXQ_ERR_CAPACITY
    float s_x;                     // per-tensor scale (per-token: the first row's)
    int32_t reserved;
};
struct ChainArgs {
    const ChainLayer *layers;      // device table
    int n_layers, M, kmax, grid;
    float tau;
    int exp_factor, qmax, cap, c, per_vec, out_kind;
    ChainResult *results;          // [n_layers] or NULL
    uint8_t *sync;                 // chain_sync_bytes(n_layers) of device memory, zero on entry: per-layer counters and maxima
    uint8_t *scratch;              // chain_scratch_bytes(...) of device memory: per-layer codes, masks, segment flags
    int32_t *dev_status;
    uint32_t spin;
    uint32_t extra_arrivals;       // test hook: a layer that waits for the one before it expects this many CTAs more
    int slots, slot_bytes;         // ring geometry
    int lgroups;                   // loader warps in use; divides slots
    int xregion;                   // bytes of the region the layers' buffers of prepared X are cut from
    const uint32_t *place;         // [n_layers] device: where in the region, and after which layers' release (chain_geometry)
};
struct ChainGeometry {
    int slots, lgroups, xregion;
};
// Fills unit_off / seg / slice_off of every entry (host copy of the table); returns the widest K, -1 if a layer
// does not fit (or the grid is too small for the slice scheme).
int chain_plan(ChainLayer *layers, int n_layers, int grid, int slot_bytes);
int chain_slot_bytes(int M);  // bytes of a ring stage for lists of M-row layers
size_t chain_sync_bytes(int n_layers);
size_t chain_scratch_bytes(const ChainLayer *layers, int n_layers, int M);
int chain_rows(int M);  // rows of codes kept per layer: M rounded up to 1, 2, 4, 8, 16
// Shared-memory geometry of a list and every layer's place in the region of prepared X; false: does not fit.
bool chain_geometry(const ChainLayer *layers, int n_layers, int M, int slot_bytes, ChainGeometry *geo, uint32_t *place);
bool chain_layer_supported(int M, int K, int N);
cudaError_t launch_decode_chain(const ChainArgs &a, cudaStream_t s);  // cooperative launch, a.grid CTAs

cudaError_t launch_mma_peak(int n, int iters, unsigned long long *cycles_out, int32_t *status, int grid,
                            cudaStream_t s);

}  // namespace muxq
