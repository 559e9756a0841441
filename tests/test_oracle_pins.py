"""Pins for the CPU oracle: it is checked against things other than itself -- a hand-worked
example, library fp16 conversion, numpy integer matmuls, exact identities of Eq. 6 / Eq. 7,
the abs-max error bound, the r = 0 reduction to textbook abs-max INT8 (Eq. 1-3), brute force
through a different arithmetic route (fp64 division, Python big ints), and metamorphic
relations.  No GPU needed."""
import numpy as np
import pytest

import muxq_synth as synth
import oracle
from conftest import load_golden


def _rand_case(seed, M, K, N, n_out=2, mult=50.0):
    x, ch = synth.make_x(seed, 7, M, K, n_out, mult, mult)
    w = synth.make_w(seed, 7, K, N)
    return x, w, ch


# ------------------------------------------------------------------ fp16 conversions
def test_f16_widening_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.f16_to_f32(int(b)) for b in bits], np.float32)
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin].view(np.uint32), ref[fin].view(np.uint32))
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))


def test_f32_to_f16_rne_matches_numpy():
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * 10.0 ** rng.integers(-8, 5, 20000),
        # exact ties between neighbouring fp16 values, normal and subnormal
        np.array([1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -25, 3 * 2.0 ** -25, 65504.0,
                  65519.9, 65520.0, 1e6, 0.0, -0.0, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -25,
                  6.1e-5, 5.96e-8, 2.9e-8, 3.0e-8], np.float64),
    ]).astype(np.float32)
    vals = np.concatenate([vals, -vals])
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f32_to_f16(float(v)) for v in vals], np.uint16)
    assert np.array_equal(got, ref)


# ------------------------------------------------------------------ hand-worked example
def test_handworked_example_exp2():
    g = load_golden("handworked_exp2.txt")
    x = g["X"].astype(np.float16)
    w = g["W"].astype(np.float16)
    assert np.array_equal(x.astype(np.float64), g["X"]) and np.array_equal(w.astype(np.float64), g["W"])
    wq, sw = oracle.quantize_weight(w)
    assert np.array_equal(wq, g["w_q"].astype(np.int8))
    assert sw[0] == np.float32(g["s_W"][0, 0])
    res = oracle.linear(x, wq, sw, tau=6.0, e=2, cap=4)
    assert res.rc == 0 and res.r == 1
    assert res.O.tolist() == g["O"].astype(int).ravel().tolist()
    assert res.s_x[0] == np.float32(g["s_X"][0, 0]) and res.s_a[0] == res.s_x[0]
    assert np.array_equal(res.body_q, g["body_q"].astype(np.int8))
    assert np.array_equal(res.aux_q, g["aux_q"].astype(np.int8))
    assert np.array_equal(res.acc_b, g["acc_b"].astype(np.int32))
    assert np.array_equal(res.acc_a, g["acc_a"].astype(np.int32))
    assert np.array_equal(res.acc, g["acc"].astype(np.int32))
    assert np.array_equal(res.y32.astype(np.float64), g["Y"])
    assert np.array_equal(res.y16.astype(np.float64), g["Y16"])


def test_handworked_example_naive():
    g = load_golden("handworked_exp2.txt")
    x = g["X"].astype(np.float16)
    wq, sw = oracle.quantize_weight(g["W"].astype(np.float16))
    res = oracle.linear(x, wq, sw, tau=1e9, e=2, cap=4)
    assert res.r == 0 and res.s_x[0] == np.float32(g["naive_s_X"][0, 0])
    assert np.array_equal(res.body_q, g["naive_x_q"].astype(np.int8))
    assert np.array_equal(res.acc, g["naive_acc"].astype(np.int32))
    assert np.array_equal(res.y32.astype(np.float64), g["naive_Y"])
    # the direction Table 1 reports: the naive error is the larger one on this example
    exact = g["X"] @ g["W"]
    assert np.abs(g["naive_Y"] - exact).sum() > np.abs(g["Y"] - exact).sum()


# ------------------------------------------------------------------ detection rule
def test_threshold_is_strict_and_sorted_and_capacity():
    x = np.zeros((3, 16), np.float16)
    x[1, 3] = 6.0      # equal to the threshold: not an outlier
    x[2, 9] = -6.004   # next fp16 above 6 in magnitude
    x[0, 12] = 100.0
    x[2, 1] = 7.0
    cm = oracle.colmax(x)
    assert cm[3] == 6.0 and cm[9] > 6.0
    O, r, rc = oracle.detect(cm, 6.0, 8)
    assert rc == 0 and r == 3 and O.tolist() == [1, 9, 12]
    O, r, rc = oracle.detect(cm, 6.0, 2)
    assert rc == oracle.ERR_CAPACITY and r == 3 and O.tolist() == [1, 9]
    wq = np.ones((16, 8), np.int8)
    res = oracle.linear(x, wq, np.ones(1, np.float32), cap=2)
    assert res.rc == oracle.ERR_CAPACITY and res.r == 3


def test_nonfinite_inputs_rejected():
    x = np.ones((2, 16), np.float16)
    x[1, 5] = np.inf
    with pytest.raises(ValueError):
        oracle.colmax(x)


# ------------------------------------------------------------------ r = 0: textbook abs-max INT8
@pytest.mark.parametrize("per_vector", [False, True])
def test_zero_outliers_reduces_to_plain_absmax_int8(per_vector):
    x, w, _ = _rand_case(3, 37, 48, 24, n_out=2)
    wq, sw = oracle.quantize_weight(w, per_channel=per_vector)
    res = oracle.linear(x, wq, sw, tau=1e9, per_vector=per_vector)
    assert res.r == 0
    # independent numpy statement of Eq. 1-3
    xf = x.astype(np.float32)
    wf = w.astype(np.float32)
    if per_vector:
        s_x = np.abs(xf).max(axis=1, keepdims=True) / np.float32(127)
        s_w = np.abs(wf).max(axis=0, keepdims=True) / np.float32(127)
    else:
        s_x = np.abs(xf).max().reshape(1, 1) / np.float32(127)
        s_w = np.abs(wf).max().reshape(1, 1) / np.float32(127)
    xq = np.rint(xf / s_x).astype(np.int32)
    wq_np = np.rint(wf / s_w).astype(np.int32)
    acc = xq @ wq_np
    y = (s_x * s_w).astype(np.float32) * acc.astype(np.float32)
    assert np.array_equal(wq.astype(np.int32), wq_np)
    assert np.array_equal(res.body_q.astype(np.int32), xq)
    assert np.array_equal(res.acc, acc) and np.array_equal(res.acc_a, np.zeros_like(acc))
    assert np.array_equal(res.y32, y)
    assert np.array_equal(res.y16, y.astype(np.float16))


@pytest.mark.parametrize("per_channel", [False, True])
@pytest.mark.parametrize("bits", [8, 7, 5, 4, 2])
def test_weight_quantization_at_reduced_bit_widths(bits, per_channel):
    """Eq. 2 with qmax = 2^(bits-1) - 1 (the W 5 / W 4 settings of Table 2), against a numpy statement of the
    same formula; the ties at 0.5 and 2.5 of the second matrix must go to the even neighbour."""
    q = (1 << (bits - 1)) - 1
    w = synth.make_w(11, 5, 96, 40)
    tie = np.zeros((4, 8), np.float16)
    tie[0, :] = q                      # abs-max = q in every column: scale exactly 1
    tie[1, :4] = [0.5, 1.5, 2.5, -0.5]
    tie[2, :4] = [-1.5, -2.5, 3.5, 0.25]
    for mat in (w, tie):
        wq, sw = oracle.quantize_weight(mat, bits=bits, per_channel=per_channel)
        f = mat.astype(np.float32)
        amax = np.abs(f).max(axis=0, keepdims=True) if per_channel else np.abs(f).max().reshape(1, 1)
        s = (amax / np.float32(q)).astype(np.float32)
        ref = np.clip(np.rint(f / s), -q, q).astype(np.int32)
        assert np.array_equal(sw, s.ravel())
        assert np.array_equal(wq.astype(np.int32), ref)
        assert np.abs(wq.astype(np.int32)).max() == q      # the abs-max element maps to +-q, nothing beyond
    if q >= 3:
        wq, _ = oracle.quantize_weight(tie, bits=bits, per_channel=per_channel)
        assert wq[1, :4].tolist() == [0, 2, 2, 0] and wq[2, :4].tolist() == [-2, -2, min(4, q), 0]


# ------------------------------------------------------------------ Eq. 6 / Eq. 7 identities
@pytest.mark.parametrize("e", [1, 2, 3])
def test_decomposition_reconstructs_x_exactly(e):
    x, w, ch = _rand_case(5, 64, 96, 40, n_out=5, mult=70.0)
    cm = oracle.colmax(x)
    O, r, rc = oracle.detect(cm, 6.0, 64)
    assert set(ch.tolist()) <= set(O.tolist())
    body, aux = oracle.decompose(x, O, e)
    c = 2 ** e - 1
    recon = body.copy()
    recon[:, O] = body[:, O] + np.float32(c) * aux          # Eq. 6, single fp32 ops
    assert np.array_equal(recon, x.astype(np.float32))
    non = np.setdiff1d(np.arange(x.shape[1]), O)
    assert np.array_equal(body[:, non], x.astype(np.float32)[:, non])
    assert np.array_equal(aux, body[:, O])                    # Eq. 5
    assert np.array_equal(body[:, O] * np.float32(2 ** e), x.astype(np.float32)[:, O])  # Eq. 4
    # Eq. 7 before quantization reproduces X.W
    wd = w.astype(np.float64)
    y = body.astype(np.float64) @ wd + c * (aux.astype(np.float64) @ wd[O])
    ref = x.astype(np.float64) @ wd
    assert np.allclose(y, ref, rtol=0, atol=1e-9 * np.abs(ref).max())


# ------------------------------------------------------------------ quantization properties
@pytest.mark.parametrize("bits", [8, 6, 5])
@pytest.mark.parametrize("per_token", [False, True])
def test_quantization_error_bound_and_range(bits, per_token):
    x, _, _ = _rand_case(11, 50, 80, 8, n_out=3)
    O, r, _ = oracle.detect(oracle.colmax(x), 6.0, 64)
    body, aux = oracle.decompose(x, O, 2)
    s_x, s_a, bq, aq = oracle.quantize_act(body, aux, bits, per_token, False)
    q = 2 ** (bits - 1) - 1
    s = s_x.reshape(-1, 1).astype(np.float64)
    amax = np.abs(body).max(axis=1, keepdims=True) if per_token else np.abs(body).max().reshape(1, 1)
    assert np.array_equal(s_x.reshape(-1, 1), (amax / np.float32(q)).astype(np.float32))
    err = np.abs(body.astype(np.float64) - s * bq.astype(np.float64))
    assert (err <= s / 2 * (1 + 2.0 ** -22)).all()
    assert bq.min() >= -q and bq.max() <= q
    # the abs-max element of each unit maps to +-q
    hit = (np.abs(body) == amax)
    assert (np.abs(bq[hit]) == q).all()
    assert np.array_equal(aq, bq[:, O])                       # shared scale: identical codes


def test_aux_own_scale_uses_aux_absmax():
    x, _, _ = _rand_case(12, 40, 64, 8, n_out=2)
    x[:, 0] = np.float16(5.5)  # Body's abs-max can now sit outside O, so the two scales differ
    O, r, _ = oracle.detect(oracle.colmax(x), 6.0, 64)
    body, aux = oracle.decompose(x, O, 2)
    for per_token in (False, True):
        s_x, s_a, bq, aq = oracle.quantize_act(body, aux, 8, per_token, True)
        am = np.abs(aux).max(axis=1) if per_token else np.abs(aux).max().reshape(1)
        assert np.array_equal(s_a, (am / np.float32(127)).astype(np.float32))
        ref = np.rint(aux / s_a.reshape(-1, 1)).astype(np.int8)
        assert np.array_equal(aq, ref)


def test_all_zero_tensor_and_row():
    x = np.zeros((4, 16), np.float16)
    wq = np.ones((16, 8), np.int8)
    res = oracle.linear(x, wq, np.ones(1, np.float32))
    assert res.s_x[0] == 1.0 and not res.body_q.any() and not res.y32.any()
    x[1, 2] = 3.0
    res = oracle.linear(x, np.ones((16, 8), np.int8), np.ones(8, np.float32), per_vector=True)
    assert res.s_x[0] == 1.0 and res.s_x[1] == np.float32(3.0) / np.float32(127)
    assert res.body_q[1, 2] == 127


# ------------------------------------------------------------------ integer identities
@pytest.mark.parametrize("e", [1, 2, 3])
def test_integer_identity_shared_scale(e):
    x, w, _ = _rand_case(21, 33, 72, 20, n_out=4, mult=60.0)
    wq, sw = oracle.quantize_weight(w)
    res = oracle.linear(x, wq, sw, e=e)
    xt = res.body_q.astype(np.int64)
    xt[:, res.O] *= 2 ** e                                    # body + (2^e - 1) aux, in codes
    ref = xt @ wq.astype(np.int64)
    assert np.array_equal(res.acc.astype(np.int64), ref)
    assert np.array_equal(res.acc_b.astype(np.int64), res.body_q.astype(np.int64) @ wq.astype(np.int64))
    assert np.array_equal(res.acc_a.astype(np.int64),
                          res.aux_q.astype(np.int64) @ wq.astype(np.int64)[res.O])


@pytest.mark.parametrize("per_vector,aux_own", [(False, False), (True, False), (False, True), (True, True)])
def test_fake_quant_cross_check(per_vector, aux_own):
    """The paper's evaluation route (quantize -> dequantize -> float matmul) in fp64."""
    x, w, _ = _rand_case(22, 41, 64, 24, n_out=3, mult=55.0)
    wq, sw = oracle.quantize_weight(w, per_channel=per_vector)
    res = oracle.linear(x, wq, sw, per_vector=per_vector, aux_own=aux_own)
    sx = res.s_x.astype(np.float64).reshape(-1, 1)
    sa = res.s_a.astype(np.float64).reshape(-1, 1)
    wdq = wq.astype(np.float64) * sw.astype(np.float64).reshape(1, -1)
    y = (sx * res.body_q) @ wdq + 3.0 * ((sa * res.aux_q) @ wdq[res.O])
    scale = np.abs(y).max()
    assert np.allclose(res.y32, y, rtol=2e-6, atol=2e-6 * scale)
    # and the whole thing approximates X.W far better than its own magnitude
    ref = x.astype(np.float64) @ w.astype(np.float64)
    assert np.linalg.norm(res.y32 - ref) < 0.1 * np.linalg.norm(ref)


# ------------------------------------------------------------------ brute force, other arithmetic route
def _brute(x, w, tau, e, per_vector):
    """Straight-line evaluation with fp64 division (innocuous double rounding for fp32
    quotients), Python round() (half to even) and Python big-int accumulation."""
    M, K = x.shape
    N = w.shape[1]
    xf = [[float(x[m, k]) for k in range(K)] for m in range(M)]
    wf = [[float(w[k, n]) for n in range(N)] for k in range(K)]
    O = [k for k in range(K) if max(abs(xf[m][k]) for m in range(M)) > tau]
    body = [[xf[m][k] / 2 ** e if k in O else xf[m][k] for k in range(K)] for m in range(M)]
    f32 = lambda v: float(np.float32(v))
    def sc(vals):
        mx = max(abs(v) for v in vals)
        return f32(mx / 127.0) if mx > 0 else 1.0
    if per_vector:
        sx = [sc(body[m]) for m in range(M)]
        sw = [sc([wf[k][n] for k in range(K)]) for n in range(N)]
    else:
        sx = [sc([v for row in body for v in row])] * M
        sw = [sc([v for row in wf for v in row])] * N
    qz = lambda v, s: max(-127, min(127, round(f32(v / s))))
    bq = [[qz(body[m][k], sx[m]) for k in range(K)] for m in range(M)]
    wq = [[qz(wf[k][n], sw[n]) for n in range(N)] for k in range(K)]
    c = 2 ** e - 1
    acc = [[sum(bq[m][k] * wq[k][n] for k in range(K)) + c * sum(bq[m][k] * wq[k][n] for k in O)
            for n in range(N)] for m in range(M)]
    y = [[f32(f32(sx[m] * sw[n]) * f32(acc[m][n])) for n in range(N)] for m in range(M)]
    return O, bq, wq, acc, y


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("per_vector", [False, True])
def test_brute_force_tiny(seed, per_vector):
    rng = np.random.default_rng(100 + seed)
    M, K, N = rng.integers(1, 9), rng.integers(1, 9), rng.integers(1, 9)
    x = (rng.standard_normal((M, K)) * 3).astype(np.float16)
    x[:, rng.integers(0, K)] *= np.float16(20.0)
    w = (rng.standard_normal((K, N)) * 0.05).astype(np.float16)
    e = int(rng.integers(1, 4))
    O, bq, wq_b, acc, y = _brute(x, w, 6.0, e, per_vector)
    wq, sw = oracle.quantize_weight(w, per_channel=per_vector)
    res = oracle.linear(x, wq, sw, e=e, per_vector=per_vector)
    assert res.O.tolist() == O
    assert res.body_q.tolist() == bq and wq.tolist() == wq_b
    assert res.acc.tolist() == acc
    assert np.array_equal(res.y32, np.array(y, np.float32).reshape(M, N))


def test_bias_is_one_fp32_addition_after_eq3():
    """The additive term of a projection: pinned through a different arithmetic route (Python floats are fp64; the
    sum of two fp32 values is exact in fp64, so rounding it once to fp32 IS the correctly rounded fp32 sum), through
    the fp16 cast of numpy, and through the special cases: a zero bias changes nothing, a bias of -y gives zero."""
    x, w, _ = _rand_case(21, 9, 64, 24)
    wq, sw = oracle.quantize_weight(w)
    base = oracle.linear(x, wq, sw)
    rng = np.random.default_rng(5)
    bias = (rng.standard_normal(24) * 0.3).astype(np.float32)
    res = oracle.linear(x, wq, sw, bias=bias)
    want = [[np.float32(float(base.y32[m, n]) + float(bias[n])) for n in range(24)] for m in range(9)]
    assert np.array_equal(res.y32, np.array(want, np.float32))
    assert np.array_equal(res.y16.view(np.uint16), np.array(want, np.float32).astype(np.float16).view(np.uint16))
    assert np.array_equal(res.acc, base.acc) and np.array_equal(res.body_q, base.body_q)
    zero = oracle.linear(x, wq, sw, bias=np.zeros(24, np.float32))
    assert np.array_equal(zero.y32, base.y32) and np.array_equal(zero.y16.view(np.uint16), base.y16.view(np.uint16))
    # row 0 cancelled exactly
    cancel = oracle.linear(x[:1], wq, sw, bias=-oracle.linear(x[:1], wq, sw).y32[0])
    assert not cancel.y32.any()


# ------------------------------------------------------------------ metamorphic relations
def test_power_of_two_scaling():
    x, w, _ = _rand_case(31, 29, 64, 16, n_out=3)
    wq, sw = oracle.quantize_weight(w)
    a = oracle.linear(x, wq, sw, tau=6.0)
    b = oracle.linear((x.astype(np.float32) * 8).astype(np.float16), wq, sw, tau=48.0)
    assert np.array_equal(a.O, b.O) and np.array_equal(a.body_q, b.body_q)
    assert np.array_equal(a.acc, b.acc) and np.array_equal(a.y32 * np.float32(8), b.y32)


def test_row_and_channel_permutations_and_row_duplication():
    x, w, _ = _rand_case(32, 24, 48, 16, n_out=3)
    wq, sw = oracle.quantize_weight(w)
    a = oracle.linear(x, wq, sw)
    rng = np.random.default_rng(1)
    pr = rng.permutation(x.shape[0])
    b = oracle.linear(x[pr], wq, sw)
    assert np.array_equal(b.y32, a.y32[pr]) and np.array_equal(b.O, a.O)
    pc = rng.permutation(x.shape[1])
    c = oracle.linear(np.ascontiguousarray(x[:, pc]), np.ascontiguousarray(wq[pc]), sw)
    assert np.array_equal(c.acc, a.acc) and np.array_equal(c.y32, a.y32)
    assert sorted(pc[c.O].tolist()) == a.O.tolist()
    d = oracle.linear(np.concatenate([x, x[3:4]]), wq, sw)
    assert np.array_equal(d.y32[:-1], a.y32) and np.array_equal(d.y32[-1], a.y32[3])


def test_row_subset_matches_full():
    x, w, _ = _rand_case(33, 40, 64, 24, n_out=3)
    wq, sw = oracle.quantize_weight(w, per_channel=True)
    full = oracle.linear(x, wq, sw, per_vector=True)
    rows = np.array([5, 0, 39, 17], np.int32)
    sub = oracle.linear(x, wq, sw, per_vector=True, rows=rows)
    assert np.array_equal(sub.acc, full.acc[rows]) and np.array_equal(sub.y32, full.y32[rows])
    assert np.array_equal(sub.y16.view(np.uint16), full.y16.view(np.uint16)[rows])


# ------------------------------------------------------------------ statistical sanity (Table 1 direction)
def test_muxq_error_below_naive_on_config0():
    spec = synth.config_layers(0)[0]
    x, ch = spec.x()
    w = spec.w()
    wq, sw = oracle.quantize_weight(w)
    mux = oracle.linear(x, wq, sw)
    naive = oracle.linear(x, wq, sw, tau=1e9)
    assert set(ch.tolist()) <= set(mux.O.tolist()) and mux.r <= len(ch) + 1
    ref = x.astype(np.float64) @ w.astype(np.float64)
    e_mux = np.linalg.norm(mux.y32 - ref)
    e_naive = np.linalg.norm(naive.y32 - ref)
    assert e_mux < 0.5 * e_naive
    # per-tensor: Body's abs-max sits in an outlier channel, so both Aux-scale readings agree
    own = oracle.linear(x, wq, sw, aux_own=True)
    assert own.s_a[0] == own.s_x[0] and np.array_equal(own.aux_q, mux.aux_q)
