"""GPU parity of the list-of-layers decode launch (muxq_chain_build / muxq_chain_run): every layer of a list
must give exactly what the oracle gives for that layer alone -- integer accumulators and fp32 outputs bit
for bit, fp16 within 1 ulp, r and the scale exact -- whatever its position in the list, although the weight
stream of later layers is already running while earlier ones are computed."""
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


def _f16_key(v):
    u = v.view(np.uint16).astype(np.int32)
    return np.where(u & 0x8000, -(u & 0x7FFF), u)


_OUT = {0: torch.float16, 1: torch.float32, 2: torch.int32}


def _make_layers(mx, shapes, M, p, seed, n_out=4, mult=40.0):
    """Returns per layer: x, w (numpy), device X, W_q, s_w."""
    out = []
    for i, (K, N) in enumerate(shapes):
        x, _ = synth.make_x(seed, 10 + i, M, K, n_out, mult, mult)
        w = synth.make_w(seed, 10 + i, K, N)
        w_q, s_w = mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
        out.append((x, w, _dev(x), w_q, s_w))
    return out


def _check_layer(mx, y, x, w, p, out_kind):
    wq_o, sw_o = oracle.quantize_weight(w, bits=p.w_bits, per_channel=p.gran == 1)
    res = oracle.linear(x, wq_o, sw_o, tau=p.threshold, e=p.exp_factor, act_bits=p.act_bits, per_vector=p.gran == 1,
                        cap=p.max_outliers)
    g = y.cpu().numpy()
    if out_kind == mx.MUXQ_OUT_ACC_I32:
        assert np.array_equal(g, res.acc)
    elif out_kind == mx.MUXQ_OUT_F32:
        assert np.array_equal(g, res.y32)
    else:
        assert np.abs(_f16_key(g) - _f16_key(res.y16)).max() <= 1
    return res


@pytest.mark.parametrize("gran", [0, 1])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 7, 16])
def test_independent_layers_match_the_oracle(mx, M, gran):
    # the four GPT-2-large projections twice over (the unit offsets rotate, the ring wraps), a narrow layer, a
    # layer whose rows are split over several ring stages (K = 8192) and one with fewer units than CTAs
    shapes = [(1280, 3840), (1280, 1280), (1280, 5120), (5120, 1280), (256, 72), (8192, 264), (1280, 3840),
              (3072, 768), (1280, 1280), (5120, 1280), (64, 8)]
    p = mx.MuxqParams(gran=gran, max_outliers=32)
    for out_kind in (mx.MUXQ_OUT_F32, mx.MUXQ_OUT_F16, mx.MUXQ_OUT_ACC_I32):
        L = _make_layers(mx, shapes, M, p, seed=300 + M)
        ys = [torch.full((M, N), -7, dtype=_OUT[out_kind], device="cuda") for (_, N) in shapes]
        chain = mx.Chain([(xd, w_q, s_w, y, 0) for (_, _, xd, w_q, s_w), y in zip(L, ys)], p, out_kind)
        chain.run()
        assert chain.read_status() == 0
        results = chain.results.cpu().numpy()
        for l, ((x, w, _, _, _), y) in enumerate(zip(L, ys)):
            res = _check_layer(mx, y, x, w, p, out_kind)
            assert results[l, 0] == res.r and results[l, 1] == 0
            assert results[l, 2] == res.s_x[:1].view(np.int32)[0]
        # a second run of the same plan gives the same bits (ring, barriers and counters start over cleanly)
        before = [y.clone() for y in ys]
        chain.run()
        assert chain.read_status() == 0
        assert all(torch.equal(b, y) for b, y in zip(before, ys))


def test_one_large_layer_more_units_than_ring_slots(mx):
    """1280 -> 20480: every CTA has 17 or 18 units, more than the ring has slots, so a unit warp that has run
    ahead must wait until the loaders have reached its stage.  Sampled columns against the oracle."""
    K, N, M = 1280, 20480, 4
    p = mx.MuxqParams(max_outliers=32)
    x, _ = synth.make_x(9, 1, M, K, 8, 60.0, 60.0)
    w = synth.make_w(9, 1, K, N)
    w_q, s_w = mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
    y = torch.zeros(M, N, dtype=torch.float32, device="cuda")
    chain = mx.Chain([(_dev(x), w_q, s_w, y, 0)], p, mx.MUXQ_OUT_F32)
    chain.run()
    assert chain.read_status() == 0
    cols = np.unique(np.concatenate([np.arange(0, N, 997), np.arange(N - 64, N), np.arange(0, 64)]))
    wq_full, sw_full = oracle.quantize_weight(w)   # the per-tensor weight scale comes from the whole matrix
    res = oracle.linear(x, np.ascontiguousarray(wq_full[:, cols]), sw_full, cap=32)
    assert np.array_equal(y.cpu().numpy()[:, cols], res.y32)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_dependent_layers_wait_for_their_input(mx, M):
    """c_fc -> mlp c_proj -> c_fc ...: every layer's X is the fp16 Y of the layer before it (no activation in
    between: the point is the hand-over).  Each layer is checked against the oracle fed with the input that
    layer actually read."""
    d = 1280
    shapes = [(d, 4 * d), (4 * d, d), (d, 4 * d), (4 * d, d), (d, d)]
    p = mx.MuxqParams(max_outliers=1024)   # a single token row flags every channel whose one value exceeds 6
    x0, _ = synth.make_x(77, 1, M, d, 6, 30.0, 30.0)
    ws = [synth.make_w(77, 20 + i, K, N) for i, (K, N) in enumerate(shapes)]
    wq = [mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(w.shape[1]))) for w in ws]
    bufs = [_dev(x0)] + [torch.zeros(M, N, dtype=torch.float16, device="cuda") for (_, N) in shapes]
    layers = [(bufs[i], wq[i][0], wq[i][1], bufs[i + 1], mx.MUXQ_LAYER_WAIT_PREV if i else 0)
              for i in range(len(shapes))]
    chain = mx.Chain(layers, p, mx.MUXQ_OUT_F16)
    for _ in range(2):
        chain.run()
        assert chain.read_status() == 0
        for i in range(len(shapes)):
            x_in = bufs[i].cpu().numpy()
            assert np.isfinite(x_in.astype(np.float32)).all()
            _check_layer(mx, bufs[i + 1], x_in, ws[i], p, mx.MUXQ_OUT_F16)


@pytest.mark.parametrize("M", [1, 2, 4, 8, 16])
def test_layers_with_more_outlier_channels_than_the_channel_list_holds(mx, M):
    """Up to 64 outlier channels the Aux term comes from a list of channels; beyond that from the masked
    64-byte segments.  100 and 300 outlier channels (and 5 for the list path next to them), both K shapes."""
    shapes = [(1280, 1280), (5120, 1280), (1280, 3840), (5120, 264)]
    n_out = [100, 300, 5, 64]
    p = mx.MuxqParams(max_outliers=512)
    L = []
    for i, ((K, N), no) in enumerate(zip(shapes, n_out)):
        x, _ = synth.make_x(40 + M, 10 + i, M, K, no, 40.0, 80.0)
        w = synth.make_w(40 + M, 10 + i, K, N)
        w_q, s_w = mx.muxq_quantize(_dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
        L.append((x, w, _dev(x), w_q, s_w))
    for out_kind in (mx.MUXQ_OUT_ACC_I32, mx.MUXQ_OUT_F32):
        ys = [torch.full((M, N), -7, dtype=_OUT[out_kind], device="cuda") for (_, N) in shapes]
        chain = mx.Chain([(xd, w_q, s_w, y, 0) for (_, _, xd, w_q, s_w), y in zip(L, ys)], p, out_kind)
        chain.run()
        assert chain.read_status() == 0
        results = chain.results.cpu().numpy()
        for l, ((x, w, _, _, _), y) in enumerate(zip(L, ys)):
            res = _check_layer(mx, y, x, w, p, out_kind)
            assert results[l, 0] == res.r
        assert results[0, 0] > 64 and results[1, 0] > 64 and results[2, 0] <= 64


@pytest.mark.parametrize("M", [1, 2, 4, 16])
def test_layers_with_an_additive_term(mx, M):
    """Every other layer of the list carries a bias (fp32 [N]): fp32 outputs bit-equal to the oracle's one-addition
    reading, fp16 within 1 ulp; the layers without one are untouched by their neighbours' terms."""
    shapes = [(1280, 1280), (5120, 264), (1280, 3840), (256, 72)]
    p = mx.MuxqParams(max_outliers=32)
    L = _make_layers(mx, shapes, M, p, seed=700 + M)
    biases = [(synth.normal(700 + M, 50 + i, N) * 0.5).astype(np.float32) if i % 2 == 0 else None
              for i, (_, N) in enumerate(shapes)]
    for out_kind in (mx.MUXQ_OUT_F32, mx.MUXQ_OUT_F16):
        ys = [torch.full((M, N), -7, dtype=_OUT[out_kind], device="cuda") for (_, N) in shapes]
        chain = mx.Chain([(xd, w_q, s_w, y, 0, None if b is None else _dev(b))
                          for (_, _, xd, w_q, s_w), y, b in zip(L, ys, biases)], p, out_kind)
        chain.run()
        assert chain.read_status() == 0
        for (x, w, _, _, _), y, b in zip(L, ys, biases):
            wq_o, sw_o = oracle.quantize_weight(w)
            res = oracle.linear(x, wq_o, sw_o, cap=32, bias=b)
            g = y.cpu().numpy()
            if out_kind == mx.MUXQ_OUT_F32:
                assert np.array_equal(g, res.y32)
            else:
                assert np.abs(_f16_key(g) - _f16_key(res.y16)).max() <= 1


def test_strided_operands(mx):
    """X, W_q and Y as views into wider buffers (row pitches larger than K / N): the bytes between the rows are
    neither read as data nor written."""
    M, p = 4, mx.MuxqParams(max_outliers=32)
    shapes = [(1280, 1280), (5120, 264), (256, 72)]
    L = _make_layers(mx, shapes, M, p, seed=900)
    layers, ys, pads = [], [], []
    for (x, w, xd, w_q, s_w), (K, N) in zip(L, shapes):
        xw = torch.full((M, K + 64), 1000.0, dtype=torch.float16, device="cuda")   # would flag channels if it were read
        xw[:, :K] = xd
        ww = torch.full((N, K + 128), 77, dtype=torch.int8, device="cuda")
        ww[:, :K] = w_q
        yw = torch.full((M, N + 24), -7.0, dtype=torch.float32, device="cuda")
        layers.append((xw[:, :K], ww[:, :K], s_w, yw[:, :N], 0))
        ys.append(yw)
    chain = mx.Chain(layers, p, mx.MUXQ_OUT_F32)
    chain.run()
    assert chain.read_status() == 0
    for (x, w, _, _, _), yw, (K, N) in zip(L, ys, shapes):
        _check_layer(mx, yw[:, :N].contiguous(), x, w, p, mx.MUXQ_OUT_F32)
        assert bool((yw[:, N:] == -7.0).all())


def test_a_layer_over_capacity_is_reported_and_the_list_goes_on(mx):
    M = 4
    shapes = [(1280, 1280), (1280, 1280), (1280, 1280)]
    p = mx.MuxqParams(max_outliers=8)
    L = _make_layers(mx, shapes, M, p, seed=5, n_out=4, mult=200.0)
    x_bad, _ = synth.make_x(5, 99, M, 1280, 40, 200.0, 200.0)   # 40 channels far above the threshold, capacity 8
    L[1] = (x_bad, L[1][1], _dev(x_bad), L[1][3], L[1][4])
    ys = [torch.zeros(M, N, dtype=torch.float32, device="cuda") for (_, N) in shapes]
    chain = mx.Chain([(xd, w_q, s_w, y, 0) for (_, _, xd, w_q, s_w), y in zip(L, ys)], p, mx.MUXQ_OUT_F32)
    chain.run()
    assert chain.read_status() == mx.MUXQ_ERR_CAPACITY
    results = chain.results.cpu().numpy()
    assert results[1, 1] == mx.MUXQ_ERR_CAPACITY and results[1, 0] > 8
    for l in (0, 2):
        assert results[l, 1] == 0
        _check_layer(mx, ys[l], L[l][0], L[l][1], p, mx.MUXQ_OUT_F32)


def test_chain_argument_errors(mx):
    p = mx.MuxqParams()
    x = torch.zeros(4, 1280, dtype=torch.float16, device="cuda")
    w_q = torch.zeros(1280, 1280, dtype=torch.int8, device="cuda")
    s_w = torch.ones(1, device="cuda")
    y = torch.zeros(4, 1280, dtype=torch.float16, device="cuda")
    with pytest.raises(mx.MuxqError) as ei:      # K not a multiple of 64
        mx.Chain([(x[:, :1040].contiguous(), w_q[:, :1040].contiguous(), s_w, y, 0)], p)
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED
    with pytest.raises(mx.MuxqError) as ei:      # the first layer has no layer before it to wait for
        mx.Chain([(x, w_q, s_w, y, mx.MUXQ_LAYER_WAIT_PREV)], p)
    assert ei.value.status == mx.MUXQ_ERR_INVALID_ARG
    with pytest.raises(mx.MuxqError) as ei:
        mx.Chain([(x, w_q, s_w, y, 0)], mx.MuxqParams(aux_scale=mx.MUXQ_AUX_OWN))
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED
    x17 = torch.zeros(17, 1280, dtype=torch.float16, device="cuda")
    y17 = torch.zeros(17, 1280, dtype=torch.float16, device="cuda")
    with pytest.raises(mx.MuxqError) as ei:
        mx.Chain([(x17, w_q, s_w, y17, 0)], p)
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED
