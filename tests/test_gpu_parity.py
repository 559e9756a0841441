"""GPU parity: every stage of the CUDA path (through the C-ABI binding) against the CPU oracle on
the same seeded inputs.  Integer results (codes, accumulators, outlier sets) and fp32 scales must
match bit for bit; fp32 outputs within 1e-5 relative; fp16 outputs within 1 ulp."""
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


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def f16_ulp_diff(a, b):
    """Distance in units of fp16 spacing between two float16 arrays (as ordered integers)."""
    def key(x):
        u = x.view(np.uint16).astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u)
    return np.abs(key(a) - key(b))


def rel_err32(y, ref):
    den = np.maximum(np.abs(ref), 1e-6 * np.abs(ref).max())
    return (np.abs(y.astype(np.float64) - ref.astype(np.float64)) / den).max()


def make_case(seed, M, K, N, n_out=4, mult=50.0, bulk="normal", bulk_scale=1.0):
    x, ch = synth.make_x(seed, 3, M, K, n_out, mult, mult, bulk, bulk_scale)
    w = synth.make_w(seed, 3, K, N)
    return x, w, ch


def run_linear(mx, x, w, p, out_kind, rows=None):
    """GPU: quantize W, run the layer; returns (Y, workspace tensors) and oracle result."""
    M, K = x.shape
    N = w.shape[1]
    wsw = mx.Workspace(mx.muxq_small_workspace_bytes(N))
    w_q, s_w = mx.muxq_quantize(dev(w), p, True, wsw)
    ws = mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p))
    ws.buf.fill_(0xA5)  # everything but the words muxq_workspace_init prepares may hold garbage
    ws.init()
    y = mx.muxq_linear(dev(x), w_q, s_w, p, ws, out_kind)
    st = mx.muxq_read_status(ws)
    return y, ws, st, w_q, s_w


def oracle_linear(x, w, p, rows=None):
    per_vec = p.gran == 1
    wq, sw = oracle.quantize_weight(w, bits=p.w_bits, per_channel=per_vec)
    res = oracle.linear(x, wq, sw, tau=p.threshold, e=p.exp_factor, act_bits=p.act_bits, per_vector=per_vec,
                        cap=p.max_outliers, rows=rows)
    return wq, sw, res


def ws_views(mx, ws, M, K, N, p):
    v = mx.muxq_workspace_view(M, K, N, p)
    b = ws.buf.cpu().numpy()
    cap = p.max_outliers
    out = {
        "col_absmax": b[v.col_absmax: v.col_absmax + 4 * K].view(np.float32),
        "outlier_idx": b[v.outlier_idx: v.outlier_idx + 4 * cap].view(np.int32),
        "n_outliers": int(b[v.n_outliers: v.n_outliers + 4].view(np.int32)[0]),
        "s_x": b[v.s_x: v.s_x + 4 * (M if p.gran == 1 else 1)].view(np.float32),
        "body_q": b[v.body_q: v.body_q + M * v.ld_body_q].view(np.int8).reshape(M, v.ld_body_q)[:, :K],
        "aux_q": b[v.aux_q: v.aux_q + M * v.aux_cols].view(np.int8).reshape(M, v.aux_cols),
        "w_aux": b[v.w_aux: v.w_aux + N * v.aux_cols].view(np.int8).reshape(N, v.aux_cols),
    }
    return out


# ------------------------------------------------------------------ K1
@pytest.mark.parametrize("M,K", [(128, 768), (1, 1280), (333, 1040), (4096, 3072), (37, 16)])
def test_detect_matches_oracle(mx, M, K):
    x, _, ch = make_case(10 + M, M, K, 8, n_out=min(5, K // 4))
    x[0, 0] = 6.0  # exactly the threshold somewhere: must not flag by itself
    cap = 64
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(K))
    ws.buf.fill_(0x5A)
    cm, idx, n = mx.muxq_detect_outliers(dev(x), 6.0, cap, ws)
    cm_o = oracle.colmax(x)
    O, r, _ = oracle.detect(cm_o, 6.0, cap)
    assert np.array_equal(cm.cpu().numpy().view(np.uint32), cm_o.view(np.uint32))
    assert int(n.item()) == r
    assert np.array_equal(idx.cpu().numpy()[:min(r, cap)], O)


def test_detect_pitched_input_and_capacity_overflow(mx):
    M, K, ld = 64, 256, 320
    x, _, _ = make_case(5, M, K, 8, n_out=12)
    xp = torch.zeros(M, ld, dtype=torch.float16, device="cuda")
    xp[:, :K] = dev(x)
    xp[:, K:] = 1000.0  # padding beyond K must be ignored
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(K))
    cm, idx, n = mx.muxq_detect_outliers(xp[:, :K], 6.0, 4, ws)
    cm_o = oracle.colmax(x)
    O, r, rc = oracle.detect(cm_o, 6.0, 4)
    assert rc == oracle.ERR_CAPACITY and r >= 12
    assert int(n.item()) == r and np.array_equal(idx.cpu().numpy(), O)
    assert np.array_equal(cm.cpu().numpy(), cm_o)


# ------------------------------------------------------------------ Eq. 4-5 in the real domain
def test_build_aux_reconstructs_x(mx):
    x, _, _ = make_case(6, 200, 512, 8, n_out=6, mult=70.0)
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(512))
    xd = dev(x)
    cm, idx, n = mx.muxq_detect_outliers(xd, 6.0, 16, ws)
    for e in (1, 2, 3):
        aux, body = mx.muxq_build_aux(xd, idx, n, e)
        O, r, _ = oracle.detect(oracle.colmax(x), 6.0, 16)
        body_o, aux_o = oracle.decompose(x, O, e)
        assert np.array_equal(body.cpu().numpy(), body_o)
        a = aux.cpu().numpy()
        assert np.array_equal(a[:, :r], aux_o) and not a[:, r:].any()
        recon = body_o.copy()
        recon[:, O] = body.cpu().numpy()[:, O] + np.float32(2 ** e - 1) * a[:, :r]   # Eq. 6
        assert np.array_equal(recon, x.astype(np.float32))


# ------------------------------------------------------------------ K5 / K2
@pytest.mark.parametrize("gran", [0, 1])
@pytest.mark.parametrize("K,N,bits", [(768, 768, 8), (1040, 200, 8), (512, 264, 5)])
def test_weight_quantization_matches_oracle(mx, gran, K, N, bits):
    w = synth.make_w(7, K * 3 + N, K, N)
    p = mx.MuxqParams(gran=gran, w_bits=bits)
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(N))
    ws.buf.fill_(0x33)
    w_q, s_w = mx.muxq_quantize(dev(w), p, True, ws)
    wq_o, sw_o = oracle.quantize_weight(w, bits=bits, per_channel=bool(gran))
    assert np.array_equal(s_w.cpu().numpy().view(np.uint32), sw_o.view(np.uint32))
    assert np.array_equal(w_q.cpu().numpy(), wq_o.T)


@pytest.mark.parametrize("gran", [0, 1])
@pytest.mark.parametrize("M,K,e,bits", [(128, 768, 2, 8), (77, 1040, 2, 8), (300, 512, 3, 6), (64, 256, 1, 8)])
def test_activation_quantization_matches_oracle(mx, gran, M, K, e, bits):
    x, _, _ = make_case(20 + M, M, K, 8, n_out=5, mult=60.0)
    x[3] = 0  # an all-zero token row (per-token scale must become 1)
    p = mx.MuxqParams(gran=gran, exp_factor=e, act_bits=bits, max_outliers=16)
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(K))
    xd = dev(x)
    cm, idx, n = mx.muxq_detect_outliers(xd, p.threshold, p.max_outliers, ws)
    body_q, aux_q, s_x = mx.muxq_quantize(xd, p, False, ws, cm, idx, n)
    O, r, _ = oracle.detect(oracle.colmax(x), 6.0, 16)
    body, aux = oracle.decompose(x, O, e)
    sx_o, sa_o, bq_o, aq_o = oracle.quantize_act(body, aux, bits, bool(gran), False)
    assert np.array_equal(s_x.cpu().numpy().view(np.uint32), sx_o.view(np.uint32))
    assert np.array_equal(body_q.cpu().numpy(), bq_o)
    c = 2 ** e - 1
    a = aux_q.cpu().numpy()
    assert a.shape[1] == mx.muxq_aux_cols(p)
    for j in range(r):
        for t in range(c):
            assert np.array_equal(a[:, c * j + t], aq_o[:, j])
    assert not a[:, c * r:].any()
    # naive quantization (no outlier handling): Eq. 1 alone
    nq, _, ns = mx.muxq_quantize(xd, p, False, ws, cm, None, None, want_aux=False)
    sx_n, _, bq_n, _ = oracle.quantize_act(x.astype(np.float32), np.zeros((M, 0), np.float32), bits, bool(gran), False)
    assert np.array_equal(ns.cpu().numpy(), sx_n) and np.array_equal(nq.cpu().numpy(), bq_n)


def test_quantization_ties_round_half_even(mx):
    """Scale 0.25 exactly and inputs on multiples of 0.125: every other value is an exact .5 tie."""
    M, K = 64, 256
    rng = np.random.default_rng(3)
    x = (rng.integers(-100, 101, (M, K)) * 0.125).astype(np.float16)
    x[0, 7] = 31.75  # abs-max -> s = 31.75 / 127 = 0.25
    p = mx.MuxqParams(threshold=1e4)
    ws = mx.Workspace(mx.muxq_small_workspace_bytes(K))
    xd = dev(x)
    cm, idx, n = mx.muxq_detect_outliers(xd, p.threshold, p.max_outliers, ws)
    body_q, _, s_x = mx.muxq_quantize(xd, p, False, ws, cm, idx, n, want_aux=False)
    assert s_x.item() == 0.25
    ref = np.rint(x.astype(np.float32) / np.float32(0.25)).astype(np.int8)  # numpy rint is half-to-even
    assert (np.abs(x.astype(np.float32) / 0.25 % 1.0) == 0.5).sum() > 1000
    assert np.array_equal(body_q.cpu().numpy(), ref)
    for gran in (0, 1):
        sx_o, _, bq_o, _ = oracle.quantize_act(x.astype(np.float32), np.zeros((M, 0), np.float32), 8, bool(gran), False)
        pq = mx.MuxqParams(threshold=1e4, gran=gran)
        bq, _, sx = mx.muxq_quantize(xd, pq, False, ws, cm, idx, n, want_aux=False)
        assert np.array_equal(sx.cpu().numpy(), sx_o) and np.array_equal(bq.cpu().numpy(), bq_o)


# ------------------------------------------------------------------ K3 alone
@pytest.mark.parametrize("M,K,N", [(128, 128, 128), (128, 256, 256), (256, 768, 768), (300, 1040, 520),
                                   (1000, 512, 1288), (128, 32, 64), (129, 4096, 264)])
def test_gemm_accumulators_bit_exact(mx, M, K, N):
    rng = np.random.default_rng(M * 7 + K + N)
    a = rng.integers(-127, 128, (M, K), dtype=np.int8)
    b = rng.integers(-127, 128, (N, K), dtype=np.int8)
    p = mx.MuxqParams()
    ws = mx.Workspace(256)
    acc = mx.muxq_gemm(dev(a), None, dev(b), None, None, p, None, None, mx.MUXQ_OUT_ACC_I32, ws)
    assert mx.muxq_read_status(ws) == 0
    ref = a.astype(np.int32) @ b.astype(np.int32).T
    assert np.array_equal(acc.cpu().numpy(), ref)


def test_gemm_worst_case_magnitudes(mx):
    M, K, N = 128, 5120, 256
    a = np.full((M, K), 127, np.int8)
    b = np.full((N, K), -127, np.int8)
    b[::2] = 127
    acc = mx.muxq_gemm(dev(a), None, dev(b), None, None, mx.MuxqParams(), None, None, 2, mx.Workspace(256))
    ref = a.astype(np.int32) @ b.astype(np.int32).T
    assert np.array_equal(acc.cpu().numpy(), ref)
    assert np.abs(ref).max() > 2 ** 24  # int32 -> fp32 must round (to nearest even) here
    sx = np.array([0.0123], np.float32); sw = np.array([0.00071], np.float32)
    y = mx.muxq_gemm(dev(a), None, dev(b), None, None, mx.MuxqParams(), dev(sx), dev(sw), 1, mx.Workspace(256))
    assert np.array_equal(y.cpu().numpy(), (sx * sw) * ref.astype(np.float32))
    # odd magnitudes above 2^24 exercise the rounding itself
    a[:, :7] = 1; b[:, :7] = 1
    b[1::2, 7] = 3
    ref = a.astype(np.int32) @ b.astype(np.int32).T
    y = mx.muxq_gemm(dev(a), None, dev(b), None, None, mx.MuxqParams(), dev(sx), dev(sw), 1, mx.Workspace(256))
    assert np.array_equal(y.cpu().numpy(), (sx * sw) * ref.astype(np.float32))
    y16 = mx.muxq_gemm(dev(a), None, dev(b), None, None, mx.MuxqParams(), dev(sx), dev(sw), 0, mx.Workspace(256))
    with np.errstate(over="ignore"):
        assert np.array_equal(y16.cpu().numpy(), ((sx * sw) * ref.astype(np.float32)).astype(np.float16))


@pytest.mark.parametrize("M,K,N", [(8192, 128, 2304), (8192, 256, 768), (8192, 128, 2048)])
def test_gemm_several_tiles_per_cta_pair_full_matrix(mx, M, K, N):
    """Full-matrix check of the persistent loop beyond its first tile: 288 / 128 / 256 output tiles over 74 CTA
    pairs give every pair 2 to 4 tiles, so the flip between the two TMEM accumulator buffers, the phase wrap of
    their barriers and the operand ring running on across tiles all decide values that are compared here.  The
    reference is a float32 matrix product: every partial sum stays below 2^24, so it is exact."""
    rng = np.random.default_rng(M + 3 * K + N)
    a = rng.integers(-127, 128, (M, K), dtype=np.int8)
    b = rng.integers(-127, 128, (N, K), dtype=np.int8)
    assert 127 * 127 * K < 2 ** 24
    ref = (a.astype(np.float32) @ b.astype(np.float32).T).astype(np.int32)
    ws = mx.Workspace(256)
    acc = mx.muxq_gemm(dev(a), None, dev(b), None, None, mx.MuxqParams(), None, None, mx.MUXQ_OUT_ACC_I32, ws)
    assert mx.muxq_read_status(ws) == 0
    assert np.array_equal(acc.cpu().numpy(), ref)


@pytest.mark.parametrize("gran", [0, 1])
def test_linear_several_tiles_per_cta_pair_full_matrix(mx, gran):
    """The same through the whole layer with an Aux block (K = 256, 6 outlier channels, 288 output tiles):
    every accumulator and every output of the 8192 x 2304 result against the oracle."""
    M, K, N = 8192, 256, 2304
    x, w, _ = make_case(77, M, K, N, n_out=6, mult=50.0)
    p = mx.MuxqParams(gran=gran, max_outliers=32)
    _, _, res = oracle_linear(x, w, p)
    assert res.r >= 6
    acc, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0 and np.array_equal(acc.cpu().numpy(), res.acc)
    y16, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
    assert st == 0 and f16_ulp_diff(y16.cpu().numpy(), res.y16).max() <= 1
    y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0 and np.array_equal(y32.cpu().numpy(), res.y32)


# ------------------------------------------------------------------ whole layer
@pytest.mark.parametrize("gran", [0, 1])
@pytest.mark.parametrize("M,K,N,n_out", [(128, 768, 768, 4), (300, 1040, 520, 7), (512, 256, 1288, 0),
                                         (1024, 1280, 1280, 21)])
def test_linear_matches_oracle(mx, gran, M, K, N, n_out):
    x, w, ch = make_case(40 + M, M, K, N, n_out=n_out, mult=50.0)
    p = mx.MuxqParams(gran=gran, max_outliers=32)
    wq_o, sw_o, res = oracle_linear(x, w, p)
    assert res.r >= n_out
    # raw accumulators
    acc, ws, st, w_q, s_w = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0
    v = ws_views(mx, ws, M, K, N, p)
    assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
    assert np.array_equal(v["col_absmax"].view(np.uint32), res.colmax.view(np.uint32))
    assert np.array_equal(v["s_x"].view(np.uint32), res.s_x.view(np.uint32))
    assert np.array_equal(v["body_q"], res.body_q)
    assert np.array_equal(w_q.cpu().numpy(), wq_o.T)
    c = 3
    for j in range(res.r):
        assert np.array_equal(v["w_aux"][:, c * j], wq_o[res.O[j]])
        assert np.array_equal(v["aux_q"][:, c * j + 2], res.aux_q[:, j])
    assert np.array_equal(acc.cpu().numpy(), res.acc)
    # fp32 and fp16 outputs
    y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0 and rel_err32(y32.cpu().numpy(), res.y32) <= 1e-5
    assert np.array_equal(y32.cpu().numpy(), res.y32)  # same operands, same two roundings
    y16, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
    assert st == 0 and f16_ulp_diff(y16.cpu().numpy(), res.y16).max() <= 1


def test_handworked_example_on_gpu(mx):
    from conftest import load_golden
    g = load_golden("handworked_exp2.txt")
    K, N = 16, 8  # the 2x4 / 4x2 example embedded in zero padding
    x = np.zeros((2, K), np.float16); x[:, :4] = g["X"]
    w = np.zeros((K, N), np.float16); w[:4, :2] = g["W"]
    p = mx.MuxqParams(max_outliers=4)
    # decode path (M = 2)
    y, ws, st, w_q, s_w = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0 and np.array_equal(y.cpu().numpy()[:, :2].astype(np.float64), g["Y"])
    # tensor-core path: repeat the two rows to M = 32
    xx = np.tile(x, (16, 1))
    acc, ws, st, _, _ = run_linear(mx, xx, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0 and np.array_equal(acc.cpu().numpy()[:2, :2], g["acc"].astype(np.int32))
    y16, _, _, _, _ = run_linear(mx, xx, w, p, mx.MUXQ_OUT_F16)
    assert np.array_equal(y16.cpu().numpy()[:2, :2].astype(np.float64), g["Y16"])


@pytest.mark.parametrize("M", [1, 2, 4, 7, 16])
@pytest.mark.parametrize("K,N", [(1280, 1280), (1280, 3840), (5120, 1280), (256, 72)])
def test_decode_matches_oracle(mx, M, K, N):
    x, w, _ = make_case(60 + M + K, M, K, N, n_out=8, mult=60.0)
    for gran in (0, 1):
        p = mx.MuxqParams(gran=gran, max_outliers=32)
        _, _, res = oracle_linear(x, w, p)
        acc, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
        assert st == 0 and np.array_equal(acc.cpu().numpy(), res.acc)
        y32, _, _, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
        assert np.array_equal(y32.cpu().numpy(), res.y32)
        y16, _, _, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
        assert f16_ulp_diff(y16.cpu().numpy(), res.y16).max() <= 1


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("M", [1, 4, 16, 64])
def test_layer_call_directly_after_its_weights_were_rewritten(mx, M):
    """W_q and s_w are rewritten by ordinary kernels (the library's weight quantization, then a device copy into the
    very buffers the layer reads) directly before the layer call on the same stream.  The layer kernels fetch weight
    tiles ahead of their programmatic wait; predecessors that do not release their dependents early -- these -- must
    still be seen in full.  Decode (M <= 16) and GEMM path."""
    K, N = 1280, 1280
    p = mx.MuxqParams(max_outliers=32)
    x, _ = synth.make_x(21, 1, M, K, 6, 50.0, 50.0)
    xd = dev(x)
    ws = mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p))
    w1, w2 = synth.make_w(21, 1, K, N), synth.make_w(22, 2, K, N, sigma=0.05)
    wsw = mx.Workspace(mx.muxq_small_workspace_bytes(N))
    w_q, s_w = mx.muxq_quantize(dev(w1), p, True, wsw)
    y1 = mx.muxq_linear(xd, w_q, s_w, p, ws, mx.MUXQ_OUT_F32)           # quantize -> layer, back to back
    wq2, sw2 = mx.muxq_quantize(dev(w2), p, True, wsw)
    for _ in range(3):
        w_q.copy_(wq2); s_w.copy_(sw2)                                   # device copies into the buffers in use ...
        y2 = mx.muxq_linear(xd, w_q, s_w, p, ws, mx.MUXQ_OUT_F32)       # ... directly followed by the layer
    assert mx.muxq_read_status(ws) == 0
    for w, y in ((w1, y1), (w2, y2)):
        _, _, res = oracle_linear(x, w, p)
        assert np.array_equal(y.cpu().numpy(), res.y32)


def test_zero_outliers_equals_naive_int8(mx):
    x, w, _ = make_case(70, 256, 512, 256, n_out=0)
    p = mx.MuxqParams(threshold=1e4)
    _, _, res = oracle_linear(x, w, p)
    assert res.r == 0
    acc, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0 and np.array_equal(acc.cpu().numpy(), res.acc)


def test_capacity_overflow_sets_status_and_stays_in_bounds(mx):
    M, K, N = 256, 512, 256
    x, w, _ = make_case(71, M, K, N, n_out=12)
    p = mx.MuxqParams(max_outliers=4)
    wsw = mx.Workspace(mx.muxq_small_workspace_bytes(N))
    w_q, s_w = mx.muxq_quantize(dev(w), p, True, wsw)
    nbytes = mx.muxq_workspace_bytes(M, K, N, p)
    ws = mx.Workspace(nbytes + 4096)
    ws.buf.fill_(0x77)  # canary behind the workspace proper
    ybuf = torch.full((M + 2, N), 1234.0, dtype=torch.float16, device="cuda")
    ws_use = mx.Workspace(0)
    ws_use.buf = ws.buf[:nbytes]
    ws_use.init()
    y = mx.muxq_linear(dev(x), w_q, s_w, p, ws_use, mx.MUXQ_OUT_F16, out=ybuf[1:M + 1])
    assert mx.muxq_read_status(ws_use) == mx.MUXQ_ERR_CAPACITY
    assert (ws.buf[nbytes:] == 0x77).all()
    assert (ybuf[0] == 1234.0).all() and (ybuf[M + 1] == 1234.0).all()
    v = ws_views(mx, ws_use, M, K, N, p)
    O, r, _ = oracle.detect(oracle.colmax(x), 6.0, 4)
    assert v["n_outliers"] == r and np.array_equal(v["outlier_idx"][:4], O)


def test_all_zero_activations(mx):
    x = np.zeros((128, 256), np.float16)
    w = synth.make_w(1, 1, 256, 128)
    for gran in (0, 1):
        y, ws, st, _, _ = run_linear(mx, x, w, mx.MuxqParams(gran=gran), mx.MUXQ_OUT_F32)
        assert st == 0 and not y.cpu().numpy().any()


def test_argument_errors(mx):
    p = mx.MuxqParams()
    ws = mx.Workspace(1 << 20)
    x = torch.zeros(32, 24, dtype=torch.float16, device="cuda")   # K % 16 != 0
    w_q = torch.zeros(64, 24, dtype=torch.int8, device="cuda")
    s_w = torch.ones(1, device="cuda")
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, p, ws)
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED
    x = torch.zeros(32, 32, dtype=torch.float16, device="cuda")
    w_q = torch.zeros(64, 32, dtype=torch.int8, device="cuda")
    small = mx.Workspace(256)
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, p, small)
    assert ei.value.status == mx.MUXQ_ERR_WORKSPACE
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, mx.MuxqParams(exp_factor=5), ws)
    assert ei.value.status == mx.MUXQ_ERR_INVALID_ARG
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, mx.MuxqParams(aux_scale=1), ws, mx.MUXQ_OUT_ACC_I32)
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED


def test_host_buffer_entry_point(mx):
    M, K, N = 256, 512, 264
    x, w, _ = make_case(80, M, K, N, n_out=3)
    p = mx.MuxqParams()
    wsw = mx.Workspace(mx.muxq_small_workspace_bytes(N))
    w_q, s_w = mx.muxq_quantize(dev(w), p, True, wsw)
    ws = mx.Workspace(mx.muxq_host_workspace_bytes(M, K, N, p, mx.MUXQ_OUT_F16))
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty(M, N, dtype=torch.float16).pin_memory()
    mx.muxq_linear_host(xh, w_q, s_w, p, ws, yh, mx.MUXQ_OUT_F16)
    assert mx.muxq_read_status(ws) == 0
    _, _, res = oracle_linear(x, w, p)
    assert f16_ulp_diff(yh.numpy(), res.y16).max() <= 1


# ------------------------------------------------------------------ full benchmark sizes
def _full_size_check(mx, spec, gran, n_rows=32, cap=32, full=False):
    """One layer at its full size through muxq_linear (the launch configuration bench.py times);
    detection results, scales and every code of the full matrix are compared.  The products are compared
    on every row (full=True) or on sample rows: one row of every 128-row block of X (so that every
    output tile of the persistent GEMM loop, whichever CTA of a pair owns it, is hit) at an offset that
    walks through the block, the edges, and seeded random rows.  Each row of the layer is independent
    once O and the scales are fixed, so the oracle computes them one by one."""
    x, _ = spec.x()
    w = spec.w()
    p = mx.MuxqParams(gran=gran, max_outliers=cap)
    rows = None
    if not full:
        rng = np.random.default_rng(spec.seed * 1000 + spec.tensor_id)
        blocks = np.arange(0, spec.M, 128)
        per_block = blocks + (blocks // 128 * 37) % 128
        rows = np.unique(np.concatenate([[0, spec.M - 1, 127, 128, spec.M // 2], per_block,
                                         rng.integers(0, spec.M, n_rows)])).astype(np.int32)
        rows = rows[rows < spec.M]
    sel = slice(None) if rows is None else rows
    wq_o, sw_o, res = oracle_linear(x, w, p, rows=rows)
    assert res.rc == 0 and res.r >= spec.n_outliers
    y16, ws, st, w_q, s_w = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
    assert st == 0
    v = ws_views(mx, ws, spec.M, spec.K, spec.N, p)
    assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
    assert np.array_equal(v["col_absmax"].view(np.uint32), res.colmax.view(np.uint32))
    assert np.array_equal(v["s_x"].view(np.uint32), res.s_x.view(np.uint32))
    assert np.array_equal(v["body_q"], res.body_q)          # every code of the full matrix
    assert np.array_equal(w_q.cpu().numpy(), wq_o.T)
    assert f16_ulp_diff(y16.cpu().numpy()[sel], res.y16).max() <= 1
    acc, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0 and np.array_equal(acc.cpu().numpy()[sel], res.acc)
    y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0 and rel_err32(y32.cpu().numpy()[sel], res.y32) <= 1e-5


def test_config0_full_matrix(mx):
    _full_size_check(mx, synth.config_layers(0)[0], 0, full=True)


@pytest.mark.parametrize("gran", [0, 1])
@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config1_full_matrix(mx, layer, gran):
    _full_size_check(mx, synth.config_layers(1)[layer], gran, full=True)


@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config2_heavy_tailed_full_size_sampled_rows(mx, layer):
    _full_size_check(mx, synth.config_layers(2)[layer], 0, cap=64)


@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config3_prefill_full_size_sampled_rows(mx, layer):
    _full_size_check(mx, synth.config_layers(3)[layer], 0)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_config3_decode_full_size(mx, M):
    for spec in synth.config_layers(3, M=M):
        x, _ = spec.x()
        w = spec.w()
        p = mx.MuxqParams(max_outliers=32)
        _, _, res = oracle_linear(x, w, p)
        y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
        assert st == 0 and np.array_equal(y32.cpu().numpy(), res.y32)
        y16, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
        assert st == 0 and f16_ulp_diff(y16.cpu().numpy(), res.y16).max() <= 1
        v = ws_views(mx, ws, spec.M, spec.K, spec.N, p)
        assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)


@pytest.mark.parametrize("n_out", [0, 2, 8, 32])
def test_config4_outlier_sweep_full_size_sampled_rows(mx, n_out):
    spec = synth.config_layers(4, n_outliers=n_out, layers=36)[35 * 4 + 2]   # last layer's c_fc, 8192 x 1280 -> 5120
    _full_size_check(mx, spec, 0, cap=64)


@pytest.mark.parametrize("linear", [0, 1, 2, 3])
@pytest.mark.parametrize("layer", [0, 17, 35])
def test_config4_first_middle_last_layer(mx, layer, linear):
    """Layers 0, 17 and 35 of the 36-layer stack, all four linears (8 outlier channels): the layers are
    independent problems (fresh X per layer), so three of them with every linear shape cover the stack's shapes
    and seeds at both ends and in the middle."""
    spec = synth.config_layers(4, n_outliers=8, layers=36)[layer * 4 + linear]
    _full_size_check(mx, spec, 0, cap=64, full=(layer == 0 and linear == 1))


@pytest.mark.parametrize("e,act_bits,w_bits,gran", [(1, 8, 8, 0), (3, 6, 5, 0), (3, 7, 4, 1), (2, 5, 8, 1)])
def test_linear_other_exp_factors_and_bit_widths(mx, e, act_bits, w_bits, gran):
    """exp factor 1 / 3 and the reduced bit widths of Tables 1-2 through the whole layer (tensor-core path
    and decode path): the Aux block then repeats each column 2^e - 1 = 1 or 7 times."""
    for M, K, N in ((384, 768, 520), (5, 1280, 264)):
        x, w, _ = make_case(300 + e + act_bits, M, K, N, n_out=5, mult=50.0)
        p = mx.MuxqParams(exp_factor=e, act_bits=act_bits, w_bits=w_bits, gran=gran, max_outliers=16)
        wq_o, sw_o, res = oracle_linear(x, w, p)
        acc, ws, st, w_q, s_w = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
        assert st == 0 and np.array_equal(w_q.cpu().numpy(), wq_o.T)
        assert np.array_equal(acc.cpu().numpy(), res.acc)
        y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
        assert st == 0 and np.array_equal(y32.cpu().numpy(), res.y32)
        y16, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F16)
        assert st == 0 and f16_ulp_diff(y16.cpu().numpy(), res.y16).max() <= 1


@pytest.mark.parametrize("M", [3, 40])
@pytest.mark.parametrize("gran", [0, 1])
def test_wide_k_takes_the_separate_kernels(mx, M, gran):
    """K beyond what the fused preparation / fused decode kernels hold (8192 channels) falls back to the
    stand-alone detect and quantize kernels; same results."""
    K, N = 8320, 136
    x, w, _ = make_case(500 + M, M, K, N, n_out=9, mult=50.0)
    p = mx.MuxqParams(gran=gran, max_outliers=32)
    _, _, res = oracle_linear(x, w, p)
    acc, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_ACC_I32)
    assert st == 0 and np.array_equal(acc.cpu().numpy(), res.acc)
    v = ws_views(mx, ws, M, K, N, p)
    assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
    assert np.array_equal(v["body_q"], res.body_q)
    y32, _, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0 and np.array_equal(y32.cpu().numpy(), res.y32)


def test_one_workspace_serves_a_sequence_of_shapes(mx):
    """The layer kernels leave the prepared words of the workspace as they found them: one
    muxq_workspace_init, then different shapes, granularities and repeats, each checked against the oracle."""
    shapes = [(300, 768, 256, 0), (300, 768, 256, 0), (64, 256, 136, 1), (520, 3072, 128, 0), (8, 512, 128, 0),
              (40, 8320, 136, 0), (300, 768, 256, 1), (1000, 1024, 264, 0)]
    big = 0
    for M, K, N, gran in shapes:
        big = max(big, mx.muxq_workspace_bytes(M, K, N, mx.MuxqParams(gran=gran)))
    ws = mx.Workspace(big)
    ws.buf.fill_(0x3C)
    ws.init()
    for i, (M, K, N, gran) in enumerate(shapes):
        p = mx.MuxqParams(gran=gran)
        x, w, _ = make_case(900 + i, M, K, N, n_out=5)
        w_q, s_w = mx.muxq_quantize(dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
        y = mx.muxq_linear(dev(x), w_q, s_w, p, ws, mx.MUXQ_OUT_F32)
        assert mx.muxq_read_status(ws) == 0
        _, _, res = oracle_linear(x, w, p)
        v = ws_views(mx, ws, M, K, N, p)
        assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O), (i, M, K, N)
        assert rel_err32(y.cpu().numpy(), res.y32) <= 1e-5, (i, M, K, N)


# ------------------------------------------------------------------ own-scale reading of the Aux quantization
@pytest.mark.parametrize("M,K,N,gran,e,n_out", [(300, 768, 256, 0, 2, 5), (300, 768, 256, 1, 2, 5), (8, 512, 128, 0, 2, 3),
                                                 (1000, 1024, 264, 0, 3, 9), (520, 3072, 128, 1, 1, 6), (64, 256, 136, 0, 2, 0)])
def test_aux_own_scale_layer_matches_oracle(mx, M, K, N, gran, e, n_out):
    """Aux quantized with its own abs-max scale (the other reading of Eq. 1 for Aux): scales, Aux codes and
    outputs against the oracle's aux_own path."""
    p = mx.MuxqParams(gran=gran, exp_factor=e, aux_scale=mx.MUXQ_AUX_OWN)
    x, w, _ = make_case(1200 + M + e, M, K, N, n_out=n_out)
    wq, sw = oracle.quantize_weight(w, bits=p.w_bits, per_channel=gran == 1)
    res = oracle.linear(x, wq, sw, tau=p.threshold, e=e, act_bits=p.act_bits, per_vector=gran == 1, aux_own=True,
                        cap=p.max_outliers)
    for out_kind in (mx.MUXQ_OUT_F32, mx.MUXQ_OUT_F16):
        y, ws, st, _, _ = run_linear(mx, x, w, p, out_kind)
        assert st == 0
        v = ws_views(mx, ws, M, K, N, p)
        view = mx.muxq_workspace_view(M, K, N, p)
        b = ws.buf.cpu().numpy()
        s_a = b[view.s_a: view.s_a + 4 * (M if gran == 1 else 1)].view(np.float32)
        assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
        assert np.array_equal(v["s_x"], res.s_x) and np.array_equal(s_a, res.s_a)
        assert np.array_equal(v["body_q"], res.body_q)
        assert np.array_equal(v["aux_q"][:, :res.r], res.aux_q) and not v["aux_q"][:, res.r:].any()
        if out_kind == mx.MUXQ_OUT_F32:
            assert rel_err32(y.cpu().numpy(), res.y32) <= 1e-5
        else:
            assert f16_ulp_diff(y.cpu().numpy(), res.y16).max() <= 1


# ------------------------------------------------------------------ the layer's additive term (muxq_linear_bias)
@pytest.mark.parametrize("M,K,N,gran", [(300, 768, 256, 0), (1000, 1024, 264, 1), (2600, 256, 776, 0), (1, 1280, 264, 0),
                                        (7, 768, 136, 1), (16, 8320, 128, 0)])
@pytest.mark.parametrize("out_kind", [0, 1])
def test_linear_with_bias(mx, M, K, N, gran, out_kind):
    """Prefill shapes (both GEMM kernels' epilogues, ragged tiles) and decode shapes (fused and two-kernel form):
    fp32 outputs bit-equal to the oracle's one-addition reading, fp16 within 1 ulp."""
    p = mx.MuxqParams(gran=gran)
    x, w, _ = make_case(1800 + M + gran, M, K, N, n_out=5, mult=50.0)
    bias = (synth.normal(1800 + M, 9, N) * 0.5).astype(np.float32)
    wq, sw = oracle.quantize_weight(w, bits=p.w_bits, per_channel=gran == 1)
    res = oracle.linear(x, wq, sw, per_vector=gran == 1, bias=bias, want_codes=False)
    w_q, s_w = mx.muxq_quantize(dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N)))
    ws = mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p))
    y = mx.muxq_linear(dev(x), w_q, s_w, p, ws, out_kind, bias=dev(bias))
    assert mx.muxq_read_status(ws) == 0
    g = y.cpu().numpy()
    if out_kind == 1:
        assert np.array_equal(g, res.y32)
    else:
        assert f16_ulp_diff(g, res.y16).max() <= 1
    # without the term the same call gives the plain layer (the epilogue's branch is off, not stale)
    y0 = mx.muxq_linear(dev(x), w_q, s_w, p, ws, mx.MUXQ_OUT_F32)
    assert np.array_equal(y0.cpu().numpy(), oracle.linear(x, wq, sw, per_vector=gran == 1, want_codes=False).y32)


def test_linear_bias_argument_errors(mx):
    p = mx.MuxqParams()
    x = torch.zeros(32, 256, dtype=torch.float16, device="cuda")
    w_q = torch.zeros(128, 256, dtype=torch.int8, device="cuda")
    s_w = torch.ones(1, device="cuda")
    bias = torch.zeros(128, device="cuda")
    ws = mx.Workspace(mx.muxq_workspace_bytes(32, 256, 128, p))
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, p, ws, mx.MUXQ_OUT_ACC_I32, bias=bias)
    assert ei.value.status == mx.MUXQ_ERR_INVALID_ARG
    pown = mx.MuxqParams(aux_scale=mx.MUXQ_AUX_OWN)
    with pytest.raises(mx.MuxqError) as ei:
        mx.muxq_linear(x, w_q, s_w, pown, mx.Workspace(mx.muxq_workspace_bytes(32, 256, 128, pown)), mx.MUXQ_OUT_F32, bias=bias)
    assert ei.value.status == mx.MUXQ_ERR_UNSUPPORTED


# ------------------------------------------------------------------ an outlier set as large as K
@pytest.mark.parametrize("M,K,N,gran", [(300, 1280, 256, 0), (300, 1280, 256, 1), (260, 5120, 136, 0), (4, 1280, 264, 0),
                                        (16, 5120, 128, 1)])
def test_every_channel_an_outlier_channel(mx, M, K, N, gran):
    """A bulk wide enough that every channel holds an element above the threshold: O is all of K (beyond 1024
    channels), Aux mirrors the whole of Body, and the layer still matches the oracle code for code."""
    p = mx.MuxqParams(gran=gran, max_outliers=K)
    x, w, _ = make_case(1700 + M + gran, M, K, N, n_out=8, mult=60.0, bulk="t4", bulk_scale=6.0 if M > 16 else 40.0)
    wq, sw = oracle.quantize_weight(w, bits=p.w_bits, per_channel=gran == 1)
    res = oracle.linear(x, wq, sw, tau=p.threshold, e=p.exp_factor, act_bits=p.act_bits, per_vector=gran == 1, cap=K)
    assert res.r > 1024 and res.r >= 0.97 * K
    y, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0
    v = ws_views(mx, ws, M, K, N, p)
    assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
    assert np.array_equal(v["s_x"], res.s_x)
    if M > 16:
        assert np.array_equal(v["body_q"], res.body_q)
        c = (1 << p.exp_factor) - 1
        assert np.array_equal(v["aux_q"][:, 0:c * res.r:c], res.aux_q)
    assert rel_err32(y.cpu().numpy(), res.y32) <= 1e-5
    acc = mx.muxq_linear(dev(x), *mx.muxq_quantize(dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N))),
                         p, mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p)), mx.MUXQ_OUT_ACC_I32)
    assert np.array_equal(acc.cpu().numpy(), res.acc)


# ------------------------------------------------------------------ many outlier channels (capacity up to 1024)
@pytest.mark.parametrize("M,K,N,gran,own", [(300, 1024, 256, 0, 0), (300, 1024, 256, 1, 0), (8, 1024, 128, 0, 0),
                                             (200, 512, 136, 0, 1)])
def test_many_outlier_channels(mx, M, K, N, gran, own):
    """Heavy-tailed activations at unit scale flag most channels (Section III-C detection on a Student-t bulk):
    with max_outliers = 1024 the layer still matches the oracle code for code."""
    p = mx.MuxqParams(gran=gran, max_outliers=1024, aux_scale=own)
    # (a few rows need a wider bulk to push most channels over the threshold)
    x, w, _ = make_case(1500 + M + gran, M, K, N, n_out=8, mult=60.0, bulk="t4", bulk_scale=1.0 if M > 16 else 4.0)
    wq, sw = oracle.quantize_weight(w, bits=p.w_bits, per_channel=gran == 1)
    res = oracle.linear(x, wq, sw, tau=p.threshold, e=p.exp_factor, act_bits=p.act_bits, per_vector=gran == 1,
                        aux_own=bool(own), cap=1024)
    assert res.r > 64  # beyond the default capacity
    y, ws, st, _, _ = run_linear(mx, x, w, p, mx.MUXQ_OUT_F32)
    assert st == 0
    v = ws_views(mx, ws, M, K, N, p)
    assert v["n_outliers"] == res.r and np.array_equal(v["outlier_idx"][:res.r], res.O)
    assert np.array_equal(v["s_x"], res.s_x)
    if M > 16:
        assert np.array_equal(v["body_q"], res.body_q)
        c = 1 if own else (1 << p.exp_factor) - 1
        assert np.array_equal(v["aux_q"][:, 0:c * res.r:c], res.aux_q)
    assert rel_err32(y.cpu().numpy(), res.y32) <= 1e-5
    if not own:
        acc = mx.muxq_linear(dev(x), *mx.muxq_quantize(dev(w), p, True, mx.Workspace(mx.muxq_small_workspace_bytes(N))),
                             p, mx.Workspace(mx.muxq_workspace_bytes(M, K, N, p)), mx.MUXQ_OUT_ACC_I32)
        assert np.array_equal(acc.cpu().numpy(), res.acc)
    # the default capacity reports the overflow instead
    p64 = mx.MuxqParams(gran=gran, aux_scale=own)
    _, ws64, st64, _, _ = run_linear(mx, x, w, p64, mx.MUXQ_OUT_F32)
    assert st64 == mx.MUXQ_ERR_CAPACITY
