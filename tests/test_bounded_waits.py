"""Every device-side wait of the library is bounded.  These tests make two of them run out -- through the
fault-injection switches of include/muxq_measure.h, which only ever make a wait wait for something that never
comes; nothing traps, faults or spins without limit -- and check what the header promises: the kernel returns,
the status word reads MUXQ_ERR_TIMEOUT, nothing is written outside the output, a workspace that saw a time-out
refuses further layer calls until muxq_workspace_init, and after that (tensor memory freed, counters cleared)
the next ordinary call is bit-exact against the oracle again."""
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


CANARY = 0x5A


def _guarded(M, N, dtype):
    """[M, N] output view in the middle of a larger buffer filled with a canary byte."""
    esz = torch.empty(0, dtype=dtype).element_size()
    pad = 4096
    raw = torch.full((pad + M * N * esz + pad,), CANARY, dtype=torch.uint8, device="cuda")
    y = raw[pad: pad + M * N * esz].view(dtype).view(M, N)
    return raw, y, pad


def _canaries_intact(raw, pad):
    r = raw.cpu().numpy()
    return bool((r[:pad] == CANARY).all() and (r[-pad:] == CANARY).all())


def test_prepare_kernel_grid_barrier_times_out_and_recovers(mx):
    M, K, N = 300, 768, 256
    x, _ = synth.make_x(5, 1, M, K, 4, 50.0, 50.0)
    w = synth.make_w(5, 1, K, N)
    p = mx.MuxqParams(max_outliers=32)
    w_q, s_w = mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
    ws = mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p))
    xd = _dev(x)
    raw, y, pad = _guarded(M, N, torch.int32)
    try:
        # the barrier expects one arrival more than there are CTAs: every CTA's bounded wait runs out
        mx.muxq_test_hooks(spin_limit=4096, prep_extra_arrivals=1)
        mx.muxq_linear(xd, w_q, s_w, p, ws, mx.MUXQ_OUT_ACC_I32, out=y)
        assert mx.muxq_read_status(ws) == mx.MUXQ_ERR_TIMEOUT
    finally:
        mx.muxq_test_hooks()
    assert _canaries_intact(raw, pad)
    # the status word is sticky, and so is the mark on the workspace: an ordinary call on it fails at once
    assert mx.muxq_read_status(ws) == mx.MUXQ_ERR_TIMEOUT
    ws.clear_status()
    mx.muxq_linear(xd, w_q, s_w, p, ws, mx.MUXQ_OUT_ACC_I32, out=y)
    assert mx.muxq_read_status(ws) == mx.MUXQ_ERR_TIMEOUT
    assert _canaries_intact(raw, pad)
    # muxq_workspace_init clears the mark and the counters the time-out left dirty
    ws.init()
    acc = mx.muxq_linear(xd, w_q, s_w, p, ws, mx.MUXQ_OUT_ACC_I32, out=y)
    assert mx.muxq_read_status(ws) == 0
    wq_o, sw_o = oracle.quantize_weight(w)
    res = oracle.linear(x, wq_o, sw_o, cap=32)
    assert np.array_equal(acc.cpu().numpy(), res.acc)
    assert _canaries_intact(raw, pad)


@pytest.mark.parametrize("skip_block", [1, 3])
def test_gemm_stage_that_is_never_filled_times_out_and_recovers(mx, skip_block):
    M, K, N = 256, 512, 256          # one 256 x 256 tile for one CTA pair, four K blocks
    rng = np.random.default_rng(11 + skip_block)
    a = rng.integers(-127, 128, (M, K), dtype=np.int8)
    b = rng.integers(-127, 128, (N, K), dtype=np.int8)
    ad, bd = _dev(a), _dev(b)
    ws = mx.Workspace(256)
    raw, y, pad = _guarded(M, N, torch.int32)
    try:
        # the producer warps of both CTAs leave out the loads of one K block: the MMA warp's wait for that stage
        # runs out, the other roles are released, copies in flight are awaited, tensor memory is freed
        mx.muxq_test_hooks(spin_limit=20000, gemm_skip_k_block=skip_block + 1)
        mx.muxq_gemm(ad, None, bd, None, None, mx.MuxqParams(), None, None, mx.MUXQ_OUT_ACC_I32, ws, out=y)
        assert mx.muxq_read_status(ws) == mx.MUXQ_ERR_TIMEOUT
    finally:
        mx.muxq_test_hooks()
    assert _canaries_intact(raw, pad)
    ref = a.astype(np.int32) @ b.astype(np.int32).T
    for _ in range(3):   # the next ordinary calls find every SM's tensor memory free and give the exact result
        ws.clear_status()
        acc = mx.muxq_gemm(ad, None, bd, None, None, mx.MuxqParams(), None, None, mx.MUXQ_OUT_ACC_I32, ws, out=y)
        assert mx.muxq_read_status(ws) == 0
        assert np.array_equal(acc.cpu().numpy(), ref)
    assert _canaries_intact(raw, pad)


def test_layer_list_wait_for_the_previous_layer_times_out_and_recovers(mx):
    """Two layers, the second reads the first one's Y.  With the hook its slice warps wait for one CTA more
    than stores that Y: their bounded wait runs out, they tell the other CTAs through the plan's abort word,
    every role of every CTA leaves, and the launch ends with MUXQ_ERR_TIMEOUT.  The first layer has been
    computed by then.  The next run of the same plan (which clears the plan's counters) is bit-exact."""
    M, d = 4, 1280
    p = mx.MuxqParams(max_outliers=1024)
    x0, _ = synth.make_x(11, 1, M, d, 6, 30.0, 30.0)
    ws = [synth.make_w(11, 20 + i, d, d) for i in range(2)]
    wq = [mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(d))) for w in ws]
    y1 = torch.zeros(M, d, dtype=torch.float16, device="cuda")
    raw, y2, pad = _guarded(M, d, torch.float16)
    y2.zero_()
    chain = mx.Chain([(_dev(x0), wq[0][0], wq[0][1], y1, 0), (y1, wq[1][0], wq[1][1], y2, mx.MUXQ_LAYER_WAIT_PREV)],
                     p, mx.MUXQ_OUT_F16)

    def f16_key(v):
        u = v.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u)

    def check(y, x_in, w):
        wq_o, sw_o = oracle.quantize_weight(w)
        res = oracle.linear(x_in, wq_o, sw_o, cap=1024)
        assert np.abs(f16_key(y.cpu().numpy()) - f16_key(res.y16)).max() <= 1

    try:
        mx.muxq_test_hooks(spin_limit=2048, prep_extra_arrivals=1)
        chain.run()
        assert chain.read_status() == mx.MUXQ_ERR_TIMEOUT
        assert _canaries_intact(raw, pad)
        check(y1, x0, ws[0])
    finally:
        mx.muxq_test_hooks()
    chain.status.zero_()
    chain.run()
    assert chain.read_status() == 0
    assert _canaries_intact(raw, pad)
    check(y1, x0, ws[0])
    check(y2, y1.cpu().numpy(), ws[1])


def test_hooks_reject_a_negative_block_index(mx):
    with pytest.raises(mx.MuxqError):
        mx.muxq_test_hooks(gemm_skip_k_block=-1)
    mx.muxq_test_hooks()
