/*
 * libmuxq -- measurement and test aids.  Not part of the method (the paper has no counterpart for any of
 * them): per-kernel timing of a layer call, the INT8 issue-rate probe that serves as a roofline
 * denominator, and the fault-injection switches with which the tests make a bounded device-side wait run
 * out.  Conventions as in muxq.h.
 */
#ifndef MUXQ_MEASURE_H
#define MUXQ_MEASURE_H

#include "muxq.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * muxq_linear that also records four caller-created CUDA events (cudaEvent_t passed as void*;
 * NULL entries are skipped) on `stream` at its kernel boundaries, for per-kernel timing:
 * events[0] at entry, [1] at the start of the fused detect + redistribute + quantize kernel (after
 * the clearing step where the shape needs one: K > 8192), [2] after that kernel, [3] after the GEMM (or decode) kernel.  When `stream`
 * is being captured into a CUDA graph the records become event-record nodes, re-recorded by every
 * replay.  Same results as muxq_linear.
 */
int muxq_linear_events(const void *X_f16, int M, int K, int ldx, const int8_t *W_q, int ldw,
                       const float *s_w, int N, const muxq_params *p, void *Y, int ldy, int out_kind,
                       void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream,
                       void *const *events);

/*
 * Measurement aid: runs `ctas` CTAs (one per SM when ctas = SM count) that each issue `iters`
 * back-to-back tcgen05.mma kind::i8 instructions of shape M128 x N(mma_n = 128 or 256) x K32 on
 * operands resident in shared memory -- the issue-bound INT8 tensor rate of the GPU as it is clocked
 * right now.  cycles_per_cta [ctas] (device, uint64) receives each CTA's SM-clock cycle count from
 * first issue to completion; time the launch with CUDA events for ops/s =
 * ctas * iters * 2 * 128 * mma_n * 32 / seconds.
 */
int muxq_int8_mma_peak(int mma_n, int iters, int ctas, unsigned long long *cycles_per_cta,
                       int32_t *dev_status, void *stream);

/*
 * Fault injection for tests.  Every device-side wait of the library is bounded: it polls a limited number
 * of times and then gives up, the kernel releases what it holds (copies in flight are awaited, tensor
 * memory is freed) and raises MUXQ_ERR_TIMEOUT in the status word.  These switches let a test take that
 * path without faulting, trapping or hanging anything:
 *   spin_limit           poll limit of the waits (0 = the kernels' own, which amount to about a second)
 *   prep_extra_arrivals  the grid barrier of the preparation kernel expects this many arrivals more than
 *                        there are CTAs, so every CTA's wait runs out; in a list of layers (muxq_chain_run) a
 *                        layer flagged MUXQ_LAYER_WAIT_PREV likewise waits for that many CTAs more than
 *                        store the layer before it
 *   gemm_skip_k_block    1 + the index of a K block whose operand loads the GEMM's producer warps leave
 *                        out (0 = none): the MMA warp's wait for that stage runs out
 * The switches are process-wide and apply to launches made after the call; NULL restores normal
 * operation.  Returns MUXQ_ERR_INVALID_ARG for a negative block index.
 */
typedef struct muxq_test_hooks_t {
    uint32_t spin_limit;
    uint32_t prep_extra_arrivals;
    int32_t gemm_skip_k_block;
} muxq_test_hooks_t;
int muxq_test_hooks(const muxq_test_hooks_t *hooks);

#ifdef __cplusplus
}
#endif
#endif /* MUXQ_MEASURE_H */
