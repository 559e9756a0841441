"""muxq_linear_decode_noalloc: the decode-shaped layer whose scratch is a fixed array inside the
library, for callers that cannot allocate device memory where they call it (a decode loop that must
not stall the device with cudaMalloc, a plug-in whose host owns all device memory, a process with a
frozen memory budget).  It must give exactly what muxq_linear gives with a caller workspace, call
after call, although every call reuses the same scratch.  Collected last on purpose: a run that
stops at the first failure has then already run every other test."""
import ctypes

import numpy as np
import pytest

import muxq_synth as synth
import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mx():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2604_04701_b200 as m
    m.lib()
    return m


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("K,N", [(1280, 3840), (8192, 264), (1040, 520)])
@pytest.mark.parametrize("gran", [0, 1])
def test_two_calls_in_a_row_match_the_workspace_entry_point_and_the_oracle(mx, gran, K, N):
    """K = 8192 is the entry point's limit (and wider than one CTA of the fused preparation kernel covers, so it
    takes the separate detection and quantization kernels); K = 1040 is not a multiple of 64, so there the
    workspace entry point runs the same two kernels instead of its fused decode kernel."""
    p = mx.MuxqParams(gran=gran, max_outliers=32)
    w = synth.make_w(91, 3, K, N)
    w_q, s_w = mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
    wq_o, sw_o = oracle.quantize_weight(w, per_channel=gran == 1)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # Second call: fewer rows, fewer and weaker outlier channels, smaller maxima -- anything the
    # first call left in the shared scratch (abs-max accumulators, outlier list, codes of rows 4..15)
    # would change the result if it were not cleared or overwritten.
    cases = [synth.make_x(91, 3, 16, K, 8, 60.0, 60.0)[0], synth.make_x(92, 4, 4, K, 2, 12.0, 12.0)[0]]
    for x in cases:
        M = x.shape[0]
        xd = _dev(x)
        res = oracle.linear(x, wq_o, sw_o, per_vector=gran == 1, cap=32)
        assert res.rc == 0
        for out_kind, dt in ((mx.MUXQ_OUT_ACC_I32, torch.int32), (mx.MUXQ_OUT_F32, torch.float32),
                             (mx.MUXQ_OUT_F16, torch.float16)):
            ws = mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p))
            ref = mx.muxq_linear(xd, w_q, s_w, p, ws, out_kind)
            assert mx.muxq_read_status(ws) == 0
            out = torch.empty(M, N, dtype=dt, device="cuda")  # the caller's own output buffer
            got = mx.muxq_linear_decode_noalloc(xd, w_q, s_w, p, status, out_kind, out=out)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            # same arithmetic: integer accumulators, fp32 and fp16 outputs all bit-equal
            assert torch.equal(got, ref)
            g = got.cpu().numpy()
            if out_kind == mx.MUXQ_OUT_ACC_I32:
                assert np.array_equal(g, res.acc)
            elif out_kind == mx.MUXQ_OUT_F32:
                assert np.array_equal(g, res.y32)
            else:
                key = lambda v: np.where(v.view(np.uint16).astype(np.int32) & 0x8000,
                                         -(v.view(np.uint16).astype(np.int32) & 0x7FFF),
                                         v.view(np.uint16).astype(np.int32))
                assert np.abs(key(g) - key(res.y16)).max() <= 1


def test_sizes_beyond_the_built_in_scratch_are_refused(mx):
    lib = mx.lib()
    p = mx.MuxqParams().c()
    fake = ctypes.c_void_p(0x10000)  # aligned and never dereferenced: the size check comes first
    call = lambda M, K: lib.muxq_linear_decode_noalloc(fake, M, K, K, fake, K, fake, 768, ctypes.byref(p), fake,
                                                       768, 0, fake, None)
    assert call(17, 768) == mx.MUXQ_ERR_STATIC_LIMIT
    assert call(4, 8192 + 16) == mx.MUXQ_ERR_STATIC_LIMIT
    assert call(0, 768) == mx.MUXQ_ERR_INVALID_ARG
    assert "scratch" in mx.muxq_status_string(mx.MUXQ_ERR_STATIC_LIMIT)
