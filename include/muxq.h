/*
 * libmuxq -- MUXQ quantized linear layer (Y = X.W with outlier-channel redistribution) for
 * NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no C++ or framework types.
 *
 * Method (paper notation): X [M,K] fp16 activations, W [K,N] fp16 weights.
 *   - outlier channel = column k of X holding at least one |x| > threshold (Section III-C);
 *     O = ascending list of such k, r = |O|.
 *   - Body = X with the columns in O multiplied by 2^-exp (Eq. 4); Aux = Body[:, O] (Eq. 5);
 *     X[:, O] = Body[:, O] + (2^exp - 1) Aux (Eq. 6).
 *   - abs-max quantization (Eq. 1, Eq. 2): s = max|.| / qmax, code = round_half_even(v / s),
 *     qmax = 2^(bits-1) - 1, codes clamped to [-qmax, qmax] and stored as int8.  An all-zero
 *     unit gets s = 1.  Granularity: per tensor, or per vector = per token (row of X) and per
 *     output channel (column of W) (Section II-A, Fig. 2).
 *   - Y = dequant( Body_q.W_q + (2^exp - 1) Aux_q.W_q[O,:] ) (Eq. 7, Eq. 3), int32 accumulation.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers unless the name says "host".  Row-major; "ld" is
 *     the row pitch in ELEMENTS.  fp16 is IEEE binary16 passed as void*.
 *   - The caller owns every buffer, including the workspace; the library allocates no device
 *     memory.  The only host state it keeps between calls is a per-device record of one-time set-up
 *     (function attributes, occupancy, SM count), guarded by a mutex: a process may drive several
 *     GPUs, each call acting on the device that is current when it is made.  `stream` is a
 *     cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls only enqueue work; nothing synchronizes except muxq_read_status and
 *     muxq_linear_host's final copy-back wait when asked.
 *   - The int return value reports what the host can see at call time (bad arguments,
 *     unsupported shapes, workspace too small, CUDA launch errors).  Data-dependent conditions
 *     (more outlier channels than the capacity, an expired bounded device-side wait) are
 *     written to the device status word; a kernel never traps and never writes out of bounds.
 *     The status word is STICKY: kernels only ever raise it (atomic max), no call clears it, so
 *     one word may collect the worst status of many enqueued calls.  Zero it yourself (a 4-byte
 *     cudaMemsetAsync) before the calls whose status you want to read.
 *   - W_q and s_w are constants of a layer.  The layer kernels are launched with programmatic
 *     stream serialization and fetch their first weight tiles BEFORE they wait for the preceding
 *     work of the stream, so W_q / s_w must not be written by a kernel that (a) directly precedes a
 *     muxq_linear call on the same stream and (b) itself releases its dependents early
 *     (cudaTriggerProgrammaticLaunchCompletion / griddepcontrol.launch_dependents).  Ordinary
 *     kernels, copies and this library's own muxq_quantize are safe predecessors: without an
 *     early trigger the layer kernel starts only once they have completed.
 *   - Inputs must be finite.  NaN/Inf give unspecified (but memory-safe) results.
 *   - Alignment: X, W, Y, workspace 16-byte aligned; K % 16 == 0; ldx % 8 == 0; N % 8 == 0.
 */
#ifndef MUXQ_H
#define MUXQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MUXQ_OK = 0,
    MUXQ_ERR_INVALID_ARG = 1,
    MUXQ_ERR_UNSUPPORTED = 2,
    MUXQ_ERR_WORKSPACE = 3,
    MUXQ_ERR_CUDA = 4,
    MUXQ_ERR_CAPACITY = 5, /* device status: r > max_outliers */
    MUXQ_ERR_TIMEOUT = 6,  /* device status: a bounded wait inside a kernel expired */
    MUXQ_ERR_STATIC_LIMIT = 7 /* muxq_linear_decode_noalloc: M or K beyond its built-in scratch */
} muxq_status;

typedef enum { MUXQ_PER_TENSOR = 0, MUXQ_PER_VECTOR = 1 /* per-token X, per-channel W */ } muxq_gran;
/* Scale of the Aux block: shared with Body (Aux_q == Body_q[:,O], integer combine) or its own
 * abs-max.  The paper does not say (Eq. 5 only states Aux = Body_outlier); shared is the default. */
typedef enum { MUXQ_AUX_SHARED = 0, MUXQ_AUX_OWN = 1 } muxq_aux_scale;
typedef enum { MUXQ_OUT_F16 = 0, MUXQ_OUT_F32 = 1, MUXQ_OUT_ACC_I32 = 2 /* raw combined accumulator */ } muxq_out;

typedef struct muxq_params {
    float threshold;  /* outlier criterion, 6.0 (Section III-C) */
    int exp_factor;   /* 1..3; the paper uses 2 (Section III-C) */
    int act_bits;     /* 2..8 (Eq. 1 uses 8) */
    int w_bits;       /* 2..8 (Eq. 2 uses 8) */
    int gran;         /* muxq_gran */
    int aux_scale;    /* muxq_aux_scale; MUXQ_AUX_OWN is taken by muxq_linear / _events / _host only */
    int max_outliers; /* capacity of O, 1..8192 (every channel of the widest X); the Aux block and its cost grow with it (aux_cols below) */
} muxq_params;

/* threshold 6, exp factor 2, 8/8 bits, per tensor, shared Aux scale, capacity 64. */
void muxq_default_params(muxq_params *p);

/* Width in bytes/columns of the Aux block in GEMM operand layout:
 * round_up((2^exp - 1) * max_outliers, 128).  0 on invalid params. */
int muxq_aux_cols(const muxq_params *p);

/* Bytes of workspace muxq_linear needs for a [M,K] x [K,N] call (0 on invalid arguments). */
size_t muxq_workspace_bytes(int M, int K, int N, const muxq_params *p);
/* Bytes of workspace muxq_detect_outliers / muxq_quantize need (small; independent of M). */
size_t muxq_small_workspace_bytes(int cols);
/* Bytes of workspace muxq_linear_host needs: muxq_workspace_bytes + device staging of X and Y. */
size_t muxq_host_workspace_bytes(int M, int K, int N, const muxq_params *p, int out_kind);

/*
 * Prepares a workspace for muxq_linear / muxq_linear_events / muxq_linear_host: enqueues on `stream`
 * a zero fill of the control block and of the abs-max accumulators of the detection step
 * (Section III-C) at its start (at most 257 KiB; fewer when workspace_bytes is smaller).  The layer
 * kernels find these words zero and put them back to zero before they finish, so that a layer call
 * carries no clearing step of its own.  Call it once after allocating the workspace, before its
 * first layer call, and again
 *   - after a layer call whose status word read MUXQ_ERR_TIMEOUT (the time-out marks the workspace:
 *     every later layer call on it fails with MUXQ_ERR_TIMEOUT at once, instead of computing on
 *     half-merged channel maxima, until this call clears the mark),
 *   - after the same memory was handed to muxq_detect_outliers or muxq_quantize as their workspace,
 *     or written by anything else.
 * One workspace may then serve any sequence of layer shapes, one call at a time (calls that share a
 * workspace must be ordered on one stream or by events).  Returns MUXQ_ERR_INVALID_ARG for a NULL
 * pointer or fewer than 256 bytes.
 */
int muxq_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/*
 * Outlier-channel detection (Section III-C: a channel with at least one element of magnitude
 * greater than `threshold`, strict).
 *   X          [M,K] fp16, pitch ldx
 *   col_absmax [K] fp32 out: max_m |X[m,k]|
 *   outlier_idx[cap] int32 out: the first min(r,cap) outlier channels, ascending
 *   n_outliers [1] int32 out: r, the true count (may exceed cap)
 *   workspace  >= muxq_small_workspace_bytes(K); contents need not be initialised
 * r > cap is not an error here; muxq_linear reports it as MUXQ_ERR_CAPACITY.
 */
int muxq_detect_outliers(const void *X_f16, int M, int K, int ldx, float threshold,
                         float *col_absmax, int32_t *outlier_idx, int32_t *n_outliers, int cap,
                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * Real-domain decomposition (Eq. 4, Eq. 5), for inspection and tests.
 *   Aux  [M, ld_aux >= cap] fp32 out: Aux[m,j] = X[m,O_j] * 2^-exp for j < min(r,cap), else 0
 *   Body [M, ld_body >= K] fp32 out, or NULL: X with the columns in O multiplied by 2^-exp
 * fp32 outputs keep Eq. 6 exact: Body[:,O] + (2^exp - 1) Aux == X[:,O] bit for bit.
 */
int muxq_build_aux(const void *X_f16, int M, int K, int ldx, const int32_t *outlier_idx,
                   const int32_t *n_outliers, int cap, int exp_factor, float *Aux, int ld_aux,
                   float *Body_or_null, int ld_body, void *stream);

/*
 * Abs-max quantization (Eq. 1 for activations, Eq. 2 for weights).
 *
 * is_weight = 1: A is W [rows=K, cols=N] fp16.  Writes W_q TRANSPOSED, [N, ld_q >= K] int8
 *   (K contiguous: the tensor-core B operand layout), scales [1] (per tensor) or [N] (per
 *   vector).  col_absmax / outlier_idx / n_outliers / Aux_q are ignored (pass NULL).
 *
 * is_weight = 0: A is X [rows=M, cols=K] fp16; fused redistribute-and-quantize (Eq. 4-5 then
 *   Eq. 1).  col_absmax [K] must hold muxq_detect_outliers' output for this X.
 *   outlier_idx/n_outliers from the same call, or both NULL for naive quantization (O empty).
 *   Writes Body_q [M, ld_q >= K] int8 and, when Aux_q != NULL, the Aux block in operand layout:
 *   Aux_q [M, ld_aux >= muxq_aux_cols(p)] with Aux_q[m, c*j + t] = Body_q[m, O_j] for j < r,
 *   t < c = 2^exp - 1 (each Aux column repeated c times so that one integer accumulation yields
 *   Body_q.W_q + c Aux_q.W_q[O,:]); remaining columns zero.  scales: [1] or [M].
 *   r > p->max_outliers: only the first max_outliers channels are treated (muxq_linear flags it).
 *
 * workspace >= muxq_small_workspace_bytes(cols).
 */
int muxq_quantize(const void *A_f16, int rows, int cols, int ld, const muxq_params *p, int is_weight,
                  const float *col_absmax, const int32_t *outlier_idx, const int32_t *n_outliers,
                  int8_t *A_q, int ld_q, int8_t *Aux_q, int ld_aux, float *scales,
                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * The integer products, weighted sum and dequantization alone (Eq. 7, Eq. 3) on already
 * quantized operands:
 *   acc[m,n] = sum_k Body_q[m,k] W_q[n,k] + sum_{i < c*min(r,cap)} Aux_q[m,i] W_aux[n,i]
 *   Y[m,n]   = (s_x[m or 0] * s_w[n or 0]) * float(acc[m,n])   (F16: then rounded to fp16)
 *   Body_q [M, ld_a >= K], Aux_q [M, ld_aux], W_q [N, ldw >= K], W_aux [N, ld_waux], all int8,
 *   pitches multiples of 16.  W_aux[n, c*j+t] = W_q[n, O_j].  Aux_q/W_aux/n_outliers may be NULL
 *   (no Aux term).  s_x has M entries if gran is per vector else 1; s_w has N or 1.
 *   Y: [M, ldy] fp16 / fp32 / int32 by out_kind (int32: the raw acc).
 *   dev_status: device int32, set to MUXQ_ERR_TIMEOUT if a bounded wait expires (else untouched).
 */
int muxq_gemm(const int8_t *Body_q, int ld_a, const int8_t *Aux_q, int ld_aux, const int8_t *W_q,
              int ldw, const int8_t *W_aux, int ld_waux, const int32_t *n_outliers, int M, int K,
              int N, const muxq_params *p, const float *s_x, const float *s_w, void *Y, int ldy,
              int out_kind, int32_t *dev_status, void *stream);

/*
 * The whole layer: detect -> redistribute + quantize -> INT8 products + Aux correction ->
 * dequantize (Section III-C, Eq. 1-7).  W_q [N, ldw] and s_w come from muxq_quantize(is_weight=1)
 * with the same params.  M > 16: one preparation kernel and one tensor-core GEMM kernel.  M <= 16:
 * the memory-bound decode path, a single kernel that streams W_q once.  Y: [M, ldy] by out_kind.
 * workspace >= muxq_workspace_bytes(M,K,N,p), prepared once by muxq_workspace_init.  dev_status: device
 * int32 (sticky, see above); kernels raise it to MUXQ_ERR_CAPACITY (r > max_outliers; Y then
 * unspecified but in bounds) or MUXQ_ERR_TIMEOUT.
 * Intermediates stay in the workspace afterwards; muxq_workspace_view locates them.  For M <= 16
 * only col_absmax, outlier_idx, n_outliers and s_x are left there (the codes never leave the SMs).
 * params.aux_scale == MUXQ_AUX_OWN (the other reading of how Eq. 1 applies to Aux: its own abs-max
 * scale s_A, per tensor or per token): Aux_q [M, r] is stored once per outlier channel and padded with
 * zeros, Y = (s_X s_W) Body_q.W_q + (2^exp - 1) (s_A s_W) Aux_q.W_q[O,:] is formed from two separately
 * dequantized fp32 products (two GEMM launches and one streaming sum, for every M; workspace grows by
 * 8 M N bytes; out_kind MUXQ_OUT_ACC_I32 and K > 8192 are MUXQ_ERR_UNSUPPORTED).  Provided for
 * completeness of the method, not tuned.
 */
int muxq_linear(const void *X_f16, int M, int K, int ldx, const int8_t *W_q, int ldw,
                const float *s_w, int N, const muxq_params *p, void *Y, int ldy, int out_kind,
                void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/*
 * muxq_linear with the layer's additive term: Y[m, n] = dequantized value of Eq. 3 + bias[n].  The GPT-2
 * projections the paper measures on (Section IV-C) carry such a term; the paper's equations end at Eq. 3, so the
 * reading here is the plain one: one fp32 addition (round to nearest) after the two multiplications of Eq. 3, then
 * the cast to the output type, fused into the epilogue of the product.  bias: device, fp32 [N], 16-byte aligned,
 * constant while the call may be in flight; NULL gives muxq_linear.  MUXQ_OUT_ACC_I32 with a bias is
 * MUXQ_ERR_INVALID_ARG (the accumulator has no scale yet), MUXQ_AUX_OWN with a bias MUXQ_ERR_UNSUPPORTED.
 * Everything else as for muxq_linear.
 */
int muxq_linear_bias(const void *X_f16, int M, int K, int ldx, const int8_t *W_q, int ldw,
                     const float *s_w, const float *bias_f32, int N, const muxq_params *p, void *Y, int ldy,
                     int out_kind, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/* Where muxq_linear leaves its intermediates inside the workspace (byte offsets). */
typedef struct muxq_ws_view {
    size_t col_absmax;  /* float [K] */
    size_t outlier_idx; /* int32 [max_outliers] */
    size_t n_outliers;  /* int32 [1] */
    size_t s_x;         /* float [1] or [M] */
    size_t body_q;      /* int8 [M, ld_body_q] */
    size_t aux_q;       /* int8 [M, aux_cols]; written up to column round_up(c * r, 32): codes, then zeros */
    size_t w_aux;       /* int8 [N, aux_cols]; likewise (the products read no column beyond that) */
    size_t s_a;         /* float [1] or [M]: the Aux scale(s), MUXQ_AUX_OWN only */
    int ld_body_q;
    int aux_cols;
} muxq_ws_view;
int muxq_workspace_view(int M, int K, int N, const muxq_params *p, muxq_ws_view *view);

/*
 * muxq_linear with X and Y in HOST memory (pinned for true asynchrony): copies X to the device,
 * runs the layer, copies Y back, all on `stream`.  W_q, s_w, workspace and dev_status stay
 * device pointers.  workspace >= muxq_host_workspace_bytes(...), prepared by muxq_workspace_init.  X_host must be dense
 * (pitch K), Y_host dense (pitch N).  Does not synchronize.
 */
int muxq_linear_host(const void *X_f16_host, int M, int K, const int8_t *W_q, int ldw,
                     const float *s_w, int N, const muxq_params *p, void *Y_host, int out_kind,
                     void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/*
 * A list of decode-shaped layers (M <= 16 token rows each) in ONE persistent launch: the same computation as
 * muxq_linear with M <= 16 for every entry (Section III-C, Eq. 1, Eq. 4-5, Eq. 7, Eq. 3), with the weight
 * stream running on across layer boundaries -- what the projections of consecutive GPT-2 blocks (Section
 * IV-C: c_attn, attention c_proj, c_fc, MLP c_proj) look like to the memory system at decode time.  A layer's
 * W_q is fetched while the layers before it are still being computed; a one-layer call cannot do that.
 *
 * muxq_layer: X [M, ldx] fp16, W_q [N, ldw] int8 and s_w from muxq_quantize(is_weight = 1), Y [M, ldy] by the
 * list's out_kind; bias: fp32 [N] added after the dequantization as in muxq_linear_bias, or NULL (must be NULL
 * with MUXQ_OUT_ACC_I32).  flags = MUXQ_LAYER_WAIT_PREV says that this layer's X is written by the layer before it
 * in the list (its Y, or memory derived from nothing else): the layer's activation work then starts only when
 * every CTA has counted its part of that Y as stored (bounded waits on counters in the plan's device memory).
 * Without the flag the layers are independent.  The activation work of a layer (Section III-C, Eq. 4, Eq. 1) is
 * done once for the grid, in slices of 64 channels, and handed to all CTAs through the plan's device memory.
 * Limits: 1 <= n_layers <= 256, M <= 16, K a multiple of 64 up to 8192, N a multiple of 8, shared Aux scale;
 * alignment as for muxq_linear.  One params / M / out_kind for the whole list.  The launch is cooperative.
 *
 * muxq_chain_build validates the list, derives the schedule (which CTA streams which rows of every W_q, which
 * warp prepares which slice of every X) into plan_host -- caller-owned HOST memory of
 * muxq_chain_plan_bytes(n_layers) bytes, which must stay valid and unchanged as long as the plan is used --
 * and enqueues the copy of it to plan_dev on `stream`.  plan_dev is caller-owned device memory, 16-byte
 * aligned, of muxq_chain_device_bytes(layers, n_layers, M) bytes (0: a K that is not a positive multiple of 64,
 * n_layers or M out of range): the table, 128 bytes of counters per layer and, per layer, the codes, the
 * outlier mask and the flags of its X (about (M + 1) K bytes).  Too small a buffer is MUXQ_ERR_WORKSPACE.
 * muxq_chain_run clears the counters and enqueues the launch.  results (device, n_layers entries, or NULL)
 * receives r, the per-tensor scale and 0 / MUXQ_ERR_CAPACITY per layer; a layer whose r exceeds max_outliers
 * leaves its Y unspecified (in bounds), raises the status word, and the list goes on.  The status word is
 * sticky as everywhere.  Runs of one plan must not overlap on the GPU (the plan holds the counters and the
 * prepared activations); runs of different plans may, as far as the device can hold their CTAs at the same
 * time.  W_q and s_w are constants of the layers: they must not be written while a run that reads them may be
 * in flight.
 */
#define MUXQ_LAYER_WAIT_PREV 1
typedef struct muxq_layer {
    const void *X_f16;
    const int8_t *W_q;
    const float *s_w;
    void *Y;
    int ldx, ldw, ldy;
    int K, N;
    int flags;
    const float *bias; /* fp32 [N] added after the dequantization (as in muxq_linear_bias), or NULL */
} muxq_layer;
typedef struct muxq_chain_result {
    int32_t n_outliers; /* r of this layer's X */
    int32_t status;     /* 0 or MUXQ_ERR_CAPACITY */
    float s_x;          /* per-tensor scale (per token: the first row's) */
    int32_t reserved;
} muxq_chain_result;
size_t muxq_chain_plan_bytes(int n_layers); /* host copy; 0 on n_layers outside 1..256 */
size_t muxq_chain_device_bytes(const muxq_layer *layers_host, int n_layers, int M);
int muxq_chain_build(const muxq_layer *layers_host, int n_layers, int M, const muxq_params *p, int out_kind,
                     void *plan_host, size_t plan_host_bytes, void *plan_dev, size_t plan_dev_bytes, void *stream);
int muxq_chain_run(const void *plan_host, void *plan_dev, muxq_chain_result *results_or_null,
                   int32_t *dev_status, void *stream);

/*
 * The decode-shaped layer without a caller-provided workspace.  (The paper has no counterpart:
 * this entry point exists for the sake of callers, not of the method.)
 *
 * Some callers cannot allocate device memory where they call the layer: a decode loop in which a
 * cudaMalloc would stall every stream of the device, a plug-in inside a host program that has
 * handed all device memory to its own pool, a process past the point where its memory budget was
 * frozen.  For them the scratch that muxq_linear takes as `workspace` is a fixed array inside the
 * library: 426,752 bytes of device memory on every GPU that loads the library, held until the
 * process exits.  It covers M <= 16 token rows and K <= 8192 input channels, any N; larger M or K
 * return MUXQ_ERR_STATIC_LIMIT and launch nothing.  The call allocates and frees nothing.
 *
 * Arguments, results, alignment rules and the device status word are those of muxq_linear with
 * M <= 16, with these limits of its own: max_outliers <= 64 (else MUXQ_ERR_INVALID_ARG), the shared
 * Aux scale only (MUXQ_AUX_OWN is MUXQ_ERR_UNSUPPORTED).  It always runs two kernels (the activation
 * preparation, then the W_q-streaming product), never muxq_linear's single fused decode kernel; the
 * arithmetic and therefore the results are the same.  The first call on each device looks up the array's
 * device address (the device must be current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents: the parts
 * that must start at zero are cleared on `stream` at the head of each call, and two calls whose
 * GPU work overlaps (different streams, or graphs replayed concurrently) race on it -- keep them
 * on one stream or order them yourself.  The intermediates are not exposed.
 */
int muxq_linear_decode_noalloc(const void *X_f16, int M, int K, int ldx, const int8_t *W_q, int ldw,
                               const float *s_w, int N, const muxq_params *p, void *Y, int ldy,
                               int out_kind, int32_t *dev_status, void *stream);

/* Synchronizes `stream` and returns the device status word (or MUXQ_ERR_CUDA). */
int muxq_read_status(const int32_t *dev_status, void *stream);

const char *muxq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MUXQ_H */
