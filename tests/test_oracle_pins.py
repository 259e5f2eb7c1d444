"""Pins for the CPU checker: each test holds it against something other than itself --
a worked example derived by hand, a closed form, an invariant the paper states, a
library routine, or brute force.  No GPU needed."""
import math
import os
from fractions import Fraction as F

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantizer_worked_examples.txt")


# ---- exact-arithmetic helpers (independent of the C code) ---------------------

def _rne(fr: F) -> int:
    fl = math.floor(fr)
    d = fr - fl
    if d > F(1, 2):
        return fl + 1
    if d < F(1, 2):
        return fl
    return fl if fl % 2 == 0 else fl + 1


def _f32(fr: F) -> F:
    """correctly rounded binary32 (normal range) of an exact rational"""
    if fr == 0:
        return F(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = math.floor(math.log2(a))
    while F(2) ** e > a:
        e -= 1
    while F(2) ** (e + 1) <= a:
        e += 1
    ulp = F(2) ** (e - 23)
    return sign * _rne(a / ulp) * ulp


def _exact_quantizer(w):
    w = [F(float(x)) for x in w]
    lo, hi = min(min(w), 0), max(max(w), 0)
    s = _f32(_f32(F(hi - lo)) / 255)          # binary32 subtract, then binary32 divide
    z = max(-128, min(127, _rne(_f32(-lo / s)) - 128))
    q = [max(-128, min(127, _rne(_f32(x / s)) + z)) for x in w]
    return s, z, q


# ---- P4: worked examples (Eq. 1-2) ---------------------------------------------

def _golden_cases():
    cases = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        ws, s_hex, z, codes = [x.strip() for x in line.split("|")]
        cases.append(([float(x) for x in ws.split()], float.fromhex(s_hex), int(z), [int(c) for c in codes.split()]))
    return cases


@pytest.mark.parametrize("w,s,z,codes", _golden_cases())
def test_worked_examples(w, s, z, codes):
    q, s_o, z_o = O.quantize_weights(np.array(w, dtype=np.float32))
    assert float(s_o) == s and z_o == z and q.tolist() == codes
    # and the fixture itself agrees with exact rational arithmetic
    s_e, z_e, q_e = _exact_quantizer(w)
    assert float(s_e) == s and z_e == z and q_e == codes


def test_near_tie_is_decided_by_the_binary32_quotient():
    """For range [0, 2] the real quotient 1 / (2/255) is the tie 127.5, but binary32 delta is a
    little above 2/255, so the binary32 quotient is 127.49999 and rounds down: code 127 - 128."""
    q, s, z = O.quantize_weights(np.array([0.5, 1.0, 2.0], dtype=np.float32))
    assert F(float(s)) > F(2, 255) and z == -128
    assert q[1] == -1


def test_random_tensors_match_exact_arithmetic():
    rng = np.random.default_rng(7)
    for _ in range(40):
        n = int(rng.integers(1, 40))
        w = (rng.standard_normal(n) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
        if rng.random() < 0.3:
            w = np.abs(w)
        q, s, z = O.quantize_weights(w)
        s_e, z_e, q_e = _exact_quantizer(w.tolist())
        assert float(s) == float(s_e) and z == z_e and q.tolist() == q_e


# ---- P1: exact round trip on a power-of-two grid --------------------------------

def test_exact_round_trip_power_of_two_grid():
    k = np.arange(-128, 128)
    w = (k * 2.0 ** -7).astype(np.float32)      # lo = -1, hi = 127/128 -> delta = 2^-7 exactly
    q, s, z = O.quantize_weights(w)
    assert float(s) == 2.0 ** -7 and z == 0
    assert q.tolist() == k.tolist()
    assert np.array_equal(O.dequantize(q, s, z), w)


def test_grid_points_round_trip_any_range():
    """Integers representable in the quantized grid round-trip exactly: quantize(dequantize(q)) == q."""
    rng = np.random.default_rng(3)
    for _ in range(50):
        lo, hi = -abs(rng.standard_normal()) * 3, abs(rng.standard_normal()) * 3
        s, z = O.affine_params(lo, hi)
        codes = np.arange(-128, 128, dtype=np.int8)
        w = O.dequantize(codes, s, z)
        q2 = np.empty_like(codes)
        O.lib().actorq_ref_quantize_weights(O._p(w), O.C.c_longlong(256), O.C.c_float(s), O.C.c_int(z), O._p(q2))
        assert np.array_equal(q2, codes)


# ---- P2 / P3: error bound and exact zero ------------------------------------------

@pytest.mark.parametrize("dist", ["normal", "positive", "negative", "heavy", "tiny"])
def test_round_trip_error_at_most_half_step(dist):
    rng = np.random.default_rng(11)
    w = rng.standard_normal(20000)
    if dist == "positive":
        w = np.abs(w) + 0.5
    elif dist == "negative":
        w = -np.abs(w) - 0.25
    elif dist == "heavy":
        w = w ** 3 * 100
    elif dist == "tiny":
        w = w * 1e-20
    w = w.astype(np.float32)
    q, s, z = O.quantize_weights(w)
    recon = float(s) * (q.astype(np.float64) - z)            # Eq. 3 in double
    err = np.abs(w.astype(np.float64) - recon)
    # delta/2 plus the binary32 rounding of W/delta (|W/delta| <= 255 -> half an ulp is 2^-17)
    assert err.max() <= float(s) * (0.5 + 2.0 ** -16)
    assert q.min() >= -128 and q.max() <= 127
    # both ends of the range are representable: the extreme weight on each side of 0 gets the end code
    if w.min() < 0:
        assert q.min() == -128
    if w.max() > 0:
        assert q.max() == 127


def test_zero_is_exact():
    rng = np.random.default_rng(5)
    for _ in range(100):
        w = (rng.standard_normal(16) * 10.0 ** rng.uniform(-4, 4)).astype(np.float32)
        w[3] = 0.0
        q, s, z = O.quantize_weights(w)
        assert q[3] == z
        assert O.dequantize(np.array([z], dtype=np.int8), s, z)[0] == 0.0


def test_range_always_contains_zero():
    assert O.tensor_range(np.array([0.5, 2.0], dtype=np.float32))[:2] == (0.0, 2.0)
    assert O.tensor_range(np.array([-3.0, -1.0], dtype=np.float32))[:2] == (-3.0, 0.0)
    s, z = O.affine_params(0.5, 2.0)
    assert z == -128
    s, z = O.affine_params(-3.0, -1.0)
    assert z == 127


def test_degenerate_and_nonfinite():
    q, s, z = O.quantize_weights(np.zeros(9, dtype=np.float32))
    assert float(s) == 1.0 and z == 0 and not q.any()
    assert O.tensor_range(np.array([1.0, np.nan], dtype=np.float32))[2]
    assert O.tensor_range(np.array([1.0, -np.inf], dtype=np.float32))[2]
    with pytest.raises(ValueError):
        O.quantize_weights(np.array([np.inf], dtype=np.float32))


def test_quantizer_is_monotone():
    rng = np.random.default_rng(2)
    w = np.sort(rng.standard_normal(5000).astype(np.float32))
    q, _, _ = O.quantize_weights(w)
    assert np.all(np.diff(q.astype(np.int32)) >= 0)


def test_four_times_smaller_broadcast():
    """int8 packing makes the broadcast 4x smaller (Section 5, quantized communication)."""
    w = np.random.default_rng(0).standard_normal((256, 67)).astype(np.float32)
    q, s, z = O.quantize_weights(w)
    assert q.nbytes * 4 == w.nbytes and q.dtype == np.int8


# ---- activations -----------------------------------------------------------------

def test_input_quantization_special_values():
    s, z = O.affine_params(-1.0, 0.9921875)                    # delta = 2^-7, z = 0
    x = np.array([0.0, np.nan, np.inf, -np.inf, 1e30, -1e30, 0.9921875, -1.0], dtype=np.float32)
    q = O.quantize_input_f32(x, s, z)
    assert q[0] == z and q[1] == z
    assert q[2] == 127 and q[4] == 127 and q[3] == -128 and q[5] == -128
    assert q[6] == 127 and q[7] == -128


def test_input_quantization_error_bound():
    rng = np.random.default_rng(9)
    x = rng.uniform(-3, 5, 10000).astype(np.float32)
    s, z = O.affine_params(-3.0, 5.0)
    q = O.quantize_input_f32(x, s, z)
    recon = float(s) * (q.astype(np.float64) - z)
    assert np.abs(recon - x).max() <= float(s) * (0.5 + 2.0 ** -14)


def test_u8_frames_are_exact():
    u = np.arange(256, dtype=np.uint8)
    q = O.quantize_input_u8(u)
    assert np.array_equal(q.astype(np.int32) + 128, u.astype(np.int32))


# ---- P5 / P6: the integer layer ---------------------------------------------------

def test_expanded_identity_matches_definition():
    rng = np.random.default_rng(1)
    for (B, K, N) in [(3, 5, 4), (7, 67, 21), (2, 300, 9)]:
        a = rng.integers(-128, 128, (B, K), dtype=np.int8)
        w = rng.integers(-128, 128, (N, K), dtype=np.int8)
        bias = rng.integers(-1000, 1000, N).astype(np.int32)
        for z_a, z_w in [(0, 0), (-128, 17), (127, -128), (-5, -77)]:
            d = O.fc_acc(a, z_a, w, z_w, bias)
            e = O.fc_acc(a, z_a, w, z_w, bias, expanded=True)
            assert np.array_equal(d, e)


def test_fc_reduces_to_integer_matmul():
    rng = np.random.default_rng(4)
    B, K, N = 6, 37, 11                                   # non-square: a transposed operand fails
    a = rng.integers(-128, 128, (B, K), dtype=np.int8)
    w = rng.integers(-128, 128, (N, K), dtype=np.int8)
    assert np.array_equal(O.fc_acc(a, 0, w, 0, None), a.astype(np.int64) @ w.astype(np.int64).T)
    z_a, z_w = -31, 44
    bias = rng.integers(-5000, 5000, N).astype(np.int32)
    ref = (a.astype(np.int64) - z_a) @ (w.astype(np.int64) - z_w).T + bias
    assert np.array_equal(O.fc_acc(a, z_a, w, z_w, bias), ref)


def test_fc_extreme_codes_fit_int32():
    K = 16384
    a = np.full((1, K), 127, dtype=np.int8)
    w = np.full((1, K), -128, dtype=np.int8)
    acc = O.fc_acc(a, -128, w, 127, np.array([-(2 ** 30)], dtype=np.int32))
    assert int(acc[0, 0]) == K * 255 * -255 - 2 ** 30


# ---- P8: convolution by brute force ------------------------------------------------

def _im2col(a, KH, KW, stride):
    B, C, H, W = a.shape
    OH, OW = (H - KH) // stride + 1, (W - KW) // stride + 1
    cols = np.empty((B, OH, OW, C * KH * KW), dtype=np.int64)
    for oh in range(OH):
        for ow in range(OW):
            cols[:, oh, ow, :] = a[:, :, oh * stride:oh * stride + KH, ow * stride:ow * stride + KW].reshape(B, -1)
    return cols


@pytest.mark.parametrize("shape", [(1, 2, 5, 5, 3, 3, 3, 1), (2, 4, 12, 12, 5, 8, 8, 4), (2, 3, 9, 7, 4, 4, 2, 2)])
def test_conv_matches_im2col_matmul(shape):
    B, C, H, W, Oc, KH, KW, stride = shape
    rng = np.random.default_rng(6)
    a = rng.integers(-128, 128, (B, C, H, W), dtype=np.int8)
    w = rng.integers(-128, 128, (Oc, C, KH, KW), dtype=np.int8)
    bias = rng.integers(-99, 99, Oc).astype(np.int32)
    z_a, z_w = -128, 9
    cols = _im2col(a.astype(np.int64) - z_a, KH, KW, stride)
    ref = cols @ (w.astype(np.int64) - z_w).reshape(Oc, -1).T + bias      # [B][OH][OW][O]
    got = O.conv_acc(a, z_a, w, stride, z_w, bias)
    assert np.array_equal(got, ref.transpose(0, 3, 1, 2))


# ---- requantize, head ----------------------------------------------------------------

def test_requantize_half_to_even_and_relu():
    acc = np.array([1, 3, 5, -1, -3, 0, 2, 1000, -1000, 2 ** 31 - 1, -2 ** 31], dtype=np.int32)
    q = O.requantize_relu(acc, np.float32(0.5), -128)
    #        0.5->0 1.5->2 2.5->2 -0.5->-0 -1.5->-2(relu->0) 0  1  500  -500  huge  -huge
    assert (q.astype(np.int32) + 128).tolist() == [0, 2, 2, 0, 0, 0, 1, 255, 0, 255, 0]
    # identity multiplier with zero-point 0: codes are clamp(acc, 0, 127)
    q = O.requantize_relu(np.array([-7, 0, 5, 127, 128, 400], dtype=np.int32), np.float32(1.0), 0)
    assert q.tolist() == [0, 0, 5, 127, 127, 127]
    # a hidden zero-point other than -128: real zero is code z_out and nothing goes below it
    q = O.requantize_relu(np.array([-50, -1, 0, 1, 300], dtype=np.int32), np.float32(1.0), -100)
    assert q.tolist() == [-100, -100, -100, -99, 127]


def test_head_and_argmax():
    acc = np.array([[0, 4, -4, 4]], dtype=np.int32)
    y = O.head_dequant(acc, np.float32(0.25), False)
    assert y.tolist() == [[0.0, 1.0, -1.0, 1.0]]
    assert O.argmax(y).tolist() == [1]                    # lowest index among equal maxima
    t = O.head_dequant(acc, np.float32(0.25), True)
    assert t[0, 0] == 0.0 and abs(t[0, 1] - math.tanh(1.0)) < 1e-7 and t[0, 2] == -t[0, 1]


def test_layer_consts():
    P, M, bq = O.layer_consts(np.float32(0.5), np.float32(0.25), np.float32(0.125),
                              np.array([1.0, -0.1875, 0.0625, 1e30], dtype=np.float32), 4)
    assert float(P) == 0.125 and float(M) == 1.0
    assert bq.tolist() == [8, -2, 0, 2 ** 30]            # -1.5 -> -2, 0.5 -> 0 (half to even), clamp
    with pytest.raises(ValueError):
        O.layer_consts(np.float32(1), np.float32(1), np.float32(1), np.array([np.nan], dtype=np.float32), 1)


# ---- P7: int8 inference against the un-quantized network on hand-sized layers --------

class _L:
    def __init__(self, w, b=None):
        self.kind, self.weight, self.bias = "fc", w, b


def _bound_forward(layers, qp, x):
    """Propagate the worst-case quantization error layer by layer (ReLU and tanh are 1-Lipschitz).
    Returns the bound on |y_int8 - y_fp| for every output of one observation x."""
    eps = np.full(x.shape, float(qp.layers[0].s_a) / 2)
    a = x.astype(np.float64)
    n = len(layers)
    for i, (l, ql) in enumerate(zip(layers, qp.layers)):
        W = np.abs(l.weight.astype(np.float64))
        s_w = float(ql.s_w)
        # |sum (a+da)(w+dw) - a w| <= |w| da + (|a| + da) |dw|, plus the rounded bias
        e_out = W @ eps + (np.abs(a) + eps).sum() * s_w / 2 + float(ql.P) / 2
        pre = l.weight.astype(np.float64) @ a + (0 if l.bias is None else l.bias.astype(np.float64))
        if i + 1 < n:
            a = np.maximum(pre, 0)
            eps = e_out + float(qp.layers[i + 1].s_a) / 2
        else:
            return e_out * (1 + 1e-6) + 1e-6
    raise AssertionError


@pytest.mark.parametrize("dims,head", [([3, 4, 2], "tanh"), ([3, 4, 2], "linear"), ([2, 5, 3, 2], "tanh"), ([4, 3], "linear")])
def test_int8_forward_close_to_fp_forward(dims, head):
    rng = np.random.default_rng(12)
    layers = [_L((rng.standard_normal((dims[i + 1], dims[i])) * dims[i] ** -0.5).astype(np.float32),
                 (rng.standard_normal(dims[i + 1]) * 0.1).astype(np.float32)) for i in range(len(dims) - 1)]
    grid = np.linspace(-1.0, 1.0, 5)
    obs = np.array(np.meshgrid(*([grid] * dims[0]))).reshape(dims[0], -1).T.astype(np.float32)   # exhaustive grid
    y_fp, inputs = O.forward_f64(layers, obs, head, "f32")
    ranges = [(float(v.min()), float(v.max())) for v in inputs]
    qp = O.quantize_policy(layers, ranges, head, "f32")
    y_q, _, _ = O.forward(qp, obs)
    for r in range(obs.shape[0]):
        bound = _bound_forward(layers, qp, obs[r])
        assert np.all(np.abs(y_q[r].astype(np.float64) - y_fp[r]) <= bound), (r, y_q[r], y_fp[r], bound)
    # and the bound is not vacuous: int8 really differs from fp, but by less than a few steps
    assert np.abs(y_q - y_fp).max() > 0


def test_forward_trace_is_consistent():
    """trace entries obey the layer recurrences (guards the sequencing code in oracle.py)"""
    rng = np.random.default_rng(13)
    layers = [_L(rng.standard_normal((6, 5)).astype(np.float32)), _L(rng.standard_normal((3, 6)).astype(np.float32))]
    obs = rng.standard_normal((9, 5)).astype(np.float32)
    _, inputs = O.forward_f64(layers, obs, "linear", "f32")
    qp = O.quantize_policy(layers, [(float(v.min()), float(v.max())) for v in inputs], "argmax", "f32")
    y, act, trace = O.forward(qp, obs)
    a0 = O.quantize_input_f32(obs, qp.layers[0].s_a, qp.layers[0].z_a)
    ref0 = (a0.astype(np.int64) - qp.layers[0].z_a) @ (qp.layers[0].w_q.astype(np.int64) - qp.layers[0].z_w).T
    assert np.array_equal(trace[0][0], ref0)
    assert qp.layers[0].z_out == qp.layers[1].z_a == -128       # post-ReLU range starts at 0
    assert np.array_equal(act, np.argmax(y, axis=1))


# ---- per-output-channel quantization (Section 3.2: per channel for convolutional layers) ------

def test_per_channel_codes_match_exact_arithmetic_row_by_row():
    rng = np.random.default_rng(40)
    w = (rng.standard_normal((6, 3, 4, 4)) * np.array([0.01, 0.1, 1, 5, 0.5, 2]).reshape(6, 1, 1, 1)).astype(np.float32)
    w[4] = np.abs(w[4])                                    # a channel without negative weights
    q, s, z = O.quantize_weights_per_channel(w)
    for n in range(6):
        es, ez, eq = _exact_quantizer(w[n].ravel())
        assert F(float(s[n])) == es and int(z[n]) == ez and q[n].ravel().tolist() == eq


def test_per_channel_is_never_coarser_and_keeps_the_half_step_bound():
    rng = np.random.default_rng(41)
    w = (rng.standard_normal((16, 40)) * rng.uniform(0.01, 3.0, (16, 1))).astype(np.float32)
    q, s, z = O.quantize_weights_per_channel(w)
    _, s_t, _ = O.quantize_weights(w)
    assert np.all(s <= s_t)
    for n in range(16):
        back = O.dequantize(q[n], s[n], int(z[n])).astype(np.float64)
        assert np.all(np.abs(w[n].astype(np.float64) - back) <= float(s[n]) * (0.5 + 2.0 ** -16))
        assert O.dequantize(np.array([z[n]], dtype=np.int8), s[n], int(z[n]))[0] == 0.0       # zero stays exact


def test_per_channel_equals_per_tensor_when_all_channels_share_one_range():
    rng = np.random.default_rng(42)
    row = rng.standard_normal(24).astype(np.float32)
    w = np.stack([rng.permutation(row) for _ in range(5)])  # every row has the tensor's min and max
    q_c, s_c, z_c = O.quantize_weights_per_channel(w)
    q_t, s_t, z_t = O.quantize_weights(w)
    assert np.array_equal(q_c, q_t) and np.all(s_c == s_t) and np.all(z_c == z_t)
    layers = [_L(w, (rng.standard_normal(5) * 0.1).astype(np.float32)), _L(rng.standard_normal((3, 5)).astype(np.float32))]
    obs = rng.standard_normal((7, 24)).astype(np.float32)
    ranges = [(-3.0, 3.0), (0.0, 9.0)]
    y_t, _, tr_t = O.forward(O.quantize_policy(layers, ranges, "tanh", "f32"), obs)
    layers[0].per_channel = True
    y_c, _, tr_c = O.forward(O.quantize_policy(layers, ranges, "tanh", "f32"), obs)
    assert np.array_equal(y_t, y_c) and np.array_equal(tr_t[0][0], tr_c[0][0]) and np.array_equal(tr_t[0][1], tr_c[0][1])


def test_per_channel_integer_layers_match_numpy():
    rng = np.random.default_rng(43)
    a = rng.integers(-128, 128, (5, 37), dtype=np.int8)
    w = rng.integers(-128, 128, (9, 37), dtype=np.int8)
    z_w = rng.integers(-128, 128, 9).astype(np.int32)
    bias = rng.integers(-500, 500, 9).astype(np.int32)
    ref = (a.astype(np.int64) - 11) @ (w.astype(np.int64) - z_w[:, None]).T + bias
    assert np.array_equal(O.fc_acc_pc(a, 11, w, z_w, bias), ref)
    B, Cc, H, Wd, Oc, KH, KW, stride = 2, 3, 9, 7, 4, 4, 2, 2
    a4 = rng.integers(-128, 128, (B, Cc, H, Wd), dtype=np.int8)
    w4 = rng.integers(-128, 128, (Oc, Cc, KH, KW), dtype=np.int8)
    z4 = rng.integers(-128, 128, Oc).astype(np.int32)
    b4 = rng.integers(-99, 99, Oc).astype(np.int32)
    cols = _im2col(a4.astype(np.int64) + 128, KH, KW, stride)
    ref4 = cols @ (w4.astype(np.int64) - z4[:, None, None, None]).reshape(Oc, -1).T + b4
    assert np.array_equal(O.conv_acc_pc(a4, -128, w4, stride, z4, b4), ref4.transpose(0, 3, 1, 2))


def test_per_channel_requantize_and_head_are_the_per_tensor_routines_channel_by_channel():
    rng = np.random.default_rng(44)
    acc = rng.integers(-200000, 200000, (3, 4, 5, 2)).astype(np.int32)           # [B][N][OH][OW]
    M = np.array([2.0 ** -9, 3.3e-3, 1.7e-4, 0.5], dtype=np.float32)
    got = O.requantize_relu_pc(acc, M, -128)
    for n in range(4):
        assert np.array_equal(got[:, n], O.requantize_relu(np.ascontiguousarray(acc[:, n]), M[n], -128))
    acc2 = rng.integers(-90000, 90000, (6, 4)).astype(np.int32)
    P = np.array([1e-4, 3e-5, 7e-4, 2e-5], dtype=np.float32)
    y = O.head_dequant_pc(acc2, P, True)
    for n in range(4):
        assert np.array_equal(y[:, n], O.head_dequant(np.ascontiguousarray(acc2[:, n]), P[n], True))


def test_per_channel_int8_forward_close_to_fp_forward():
    """The propagated quantization bound with each row's own delta; and with rows of very different
    magnitude the per-channel policy is the closer one to the un-quantized network."""
    rng = np.random.default_rng(45)
    dims = [3, 6, 2]
    scale = np.array([0.02, 0.1, 0.5, 1.0, 3.0, 8.0]).reshape(6, 1)
    layers = [_L((rng.standard_normal((6, 3)) * scale).astype(np.float32), (rng.standard_normal(6) * 0.1).astype(np.float32)),
              _L((rng.standard_normal((2, 6)) / scale.T * 0.3).astype(np.float32))]
    grid = np.linspace(-1.0, 1.0, 7)
    obs = np.array(np.meshgrid(*([grid] * dims[0]))).reshape(dims[0], -1).T.astype(np.float32)
    y_fp, inputs = O.forward_f64(layers, obs, "linear", "f32")
    ranges = [(float(v.min()), float(v.max())) for v in inputs]
    y_t, _, _ = O.forward(O.quantize_policy(layers, ranges, "linear", "f32"), obs)
    for l in layers:
        l.per_channel = True
    qp = O.quantize_policy(layers, ranges, "linear", "f32")
    y_c, _, _ = O.forward(qp, obs)
    for r in range(obs.shape[0]):
        eps = np.full(3, float(qp.layers[0].s_a) / 2)
        a = obs[r].astype(np.float64)
        for i, (l, ql) in enumerate(zip(layers, qp.layers)):
            Wa = np.abs(l.weight.astype(np.float64))
            e_out = Wa @ eps + (np.abs(a) + eps).sum() * ql.s_w.astype(np.float64) / 2 + ql.P.astype(np.float64) / 2
            pre = l.weight.astype(np.float64) @ a + (0 if l.bias is None else l.bias.astype(np.float64))
            if i == 0:
                a = np.maximum(pre, 0)
                eps = e_out + float(qp.layers[1].s_a) / 2
        assert np.all(np.abs(y_c[r].astype(np.float64) - y_fp[r]) <= e_out * (1 + 1e-6) + 1e-6)
    assert np.abs(y_c - y_fp).mean() < np.abs(y_t - y_fp).mean()


# ---- actor exploration noise (Section 5, set-up) -------------------------------------------------

def test_explore_closed_forms():
    y = np.array([[0.5, -0.25, 0.75], [0.9, -0.9, 0.0]], dtype=np.float32)
    eps = np.array([[1.0, -2.0, 0.5], [4.0, -4.0, 0.0]], dtype=np.float32)
    assert np.array_equal(O.explore(y, np.zeros(2, np.float32), eps), y)                          # sigma 0: the policy's action
    got = O.explore(y, np.array([0.125, 0.25], np.float32), eps)                                  # exact in binary32
    assert np.array_equal(got, np.array([[0.625, -0.5, 0.8125], [1.0, -1.0, 0.0]], dtype=np.float32))   # second row clips
    # two roundings (product, then sum), not a fused multiply-add
    s, e, y1 = np.float32(0.1), np.float32(0.3), np.float32(1e-3)
    want = np.float32(y1 + np.float32(s * e))
    assert O.explore(np.array([[y1]]), np.array([s]), np.array([[e]]))[0, 0] == want
    rng = np.random.default_rng(3)
    out = O.explore(np.tanh(rng.standard_normal((50, 4))).astype(np.float32), rng.uniform(0, 0.2, 50).astype(np.float32),
                    rng.standard_normal((50, 4)).astype(np.float32) * 10)
    assert out.min() >= -1.0 and out.max() <= 1.0


# ---- input quantizer: the tie rule (round half to even, Eq. 1 on activations) ------------------

def test_input_quantization_ties_go_to_even():
    """delta = 2^-7 exactly, so x = (k + 1/2) * delta is an exact tie in binary32: the code is the even
    neighbour (round-half-away would give +-1, +-2, +-3)."""
    s, z = O.affine_params(-1.0, 0.9921875)
    assert float(s) == 2.0 ** -7 and z == 0
    d = 2.0 ** -7
    x = np.array([0.5 * d, -0.5 * d, 1.5 * d, -1.5 * d, 2.5 * d, -2.5 * d, 3.5 * d, -3.5 * d, 126.5 * d, -127.5 * d],
                 dtype=np.float32)
    assert O.quantize_input_f32(x, s, z).tolist() == [0, 0, 2, -2, 2, -2, 4, -4, 126, -128]
    # with a zero-point: the tie is decided before the offset is added (code = rne(x/delta) + z)
    s2, z2 = O.affine_params(0.0, 255 * d)
    assert float(s2) == d and z2 == -128
    x2 = np.array([0.5 * d, 1.5 * d, 2.5 * d, 254.5 * d], dtype=np.float32)
    assert O.quantize_input_f32(x2, s2, z2).tolist() == [-128, -126, -126, 126]


# ---- a convolutional policy through the whole sequencing code --------------------------------

class _C:
    def __init__(self, w, b, stride, in_hw):
        self.kind, self.weight, self.bias, self.stride, self.in_hw = "conv", w, b, stride, in_hw


def _conv_f64_im2col(x, w, b, stride):
    """float64 convolution by explicit patch extraction + matmul (independent of the C loops)."""
    B, Cc, H, W = x.shape
    Oc, _, KH, KW = w.shape
    OH, OW = (H - KH) // stride + 1, (W - KW) // stride + 1
    cols = np.empty((B, OH, OW, Cc * KH * KW), dtype=np.float64)
    for oh in range(OH):
        for ow in range(OW):
            cols[:, oh, ow, :] = x[:, :, oh * stride:oh * stride + KH, ow * stride:ow * stride + KW].reshape(B, -1)
    y = cols @ w.astype(np.float64).reshape(Oc, -1).T + (0 if b is None else b.astype(np.float64))
    return y.transpose(0, 3, 1, 2)


@pytest.mark.parametrize("stride,per_channel", [(1, False), (2, False), (1, True)])
def test_tiny_conv_policy_end_to_end(stride, per_channel):
    """uint8 frames 2x6x6 -> conv 3@3x3 -> FC 4 -> 2 Q-values through quantize_policy / forward.
    Holds: the u8 activation parameters, the conv accumulators against im2col + numpy int64, the
    (c, h, w) flatten into the first FC against an explicit index loop, the f64 conv against an
    im2col product, and the int8 outputs against the un-quantized network within the propagated bound."""
    rng = np.random.default_rng(50 + stride)
    Cc, H, W, Oc, KH = 2, 6, 6, 3, 3
    OH = (H - KH) // stride + 1
    w0 = (rng.standard_normal((Oc, Cc, KH, KH)) * (2.0 / (Cc * KH * KH)) ** 0.5).astype(np.float32)
    b0 = (rng.standard_normal(Oc) * 0.05).astype(np.float32)
    feat = Oc * OH * OH
    w1 = (rng.standard_normal((4, feat)) * (2.0 / feat) ** 0.5).astype(np.float32)
    b1 = (rng.standard_normal(4) * 0.05).astype(np.float32)
    w2 = (rng.standard_normal((2, 4)) * 0.7).astype(np.float32)
    layers = [_C(w0, b0, stride, (H, W)), _L(w1, b1), _L(w2, None)]
    if per_channel:
        layers[0].per_channel = True
    obs = rng.integers(0, 256, (40, Cc, H, W), dtype=np.uint8)
    obs[0] = 0
    obs[1] = 255

    # un-quantized network: the C conv loop against an im2col matmul, then the rest by numpy
    y_fp, inputs = O.forward_f64(layers, obs, "argmax", "u8")
    x0 = obs.astype(np.float64) / 255.0
    c_ref = np.maximum(_conv_f64_im2col(x0, w0, b0, stride), 0)
    assert np.allclose(inputs[1].reshape(c_ref.shape), c_ref, rtol=1e-13, atol=1e-13)
    h_ref = np.maximum(c_ref.reshape(40, -1) @ w1.astype(np.float64).T + b1, 0)
    assert np.allclose(y_fp, h_ref @ w2.astype(np.float64).T, rtol=1e-12, atol=1e-12)

    ranges = [(0.0, 1.0)] + [(float(v.min()), float(v.max())) for v in inputs[1:]]
    qp = O.quantize_policy(layers, ranges, "argmax", "u8")
    l0, l1 = qp.layers[0], qp.layers[1]
    assert float(l0.s_a) == float(np.float32(1.0) / np.float32(255.0)) and l0.z_a == -128      # u8 frames mean u/255
    y_q, act, trace = O.forward(qp, obs)

    # conv accumulators: im2col + int64 matmul on (u - 128) - z_a = u
    cols = _im2col(obs.astype(np.int64), KH, KH, stride)
    zw = np.asarray(l0.z_w, dtype=np.int64).reshape(-1, 1) if per_channel else int(l0.z_w)
    ref0 = cols @ (l0.w_q.astype(np.int64).reshape(Oc, -1) - zw).T + l0.bias_q
    assert np.array_equal(trace[0][0], ref0.transpose(0, 3, 1, 2))
    # flatten order into the FC: feature index = (c * OH + h) * OW + w
    a1 = trace[0][1]
    assert a1.shape == (40, Oc, OH, OH)
    acc1 = np.zeros((40, 4), dtype=np.int64)
    for c in range(Oc):
        for h in range(OH):
            for w_ in range(OH):
                k = (c * OH + h) * OH + w_
                acc1 += np.outer(a1[:, c, h, w_].astype(np.int64) - l1.z_a, l1.w_q[:, k].astype(np.int64) - int(l1.z_w))
    assert np.array_equal(trace[1][0], acc1 + l1.bias_q)
    assert np.array_equal(act, np.argmax(y_q, axis=1))

    # propagated quantization bound, layer by layer (frames are exact: eps_0 = 0)
    for r in range(40):
        a = x0[r].reshape(1, Cc, H, W)
        eps = np.zeros_like(a)
        sw0 = (np.asarray(l0.s_w, dtype=np.float64).reshape(-1, 1, 1) if per_channel else float(l0.s_w))
        P0 = (np.asarray(l0.P, dtype=np.float64).reshape(-1, 1, 1) if per_channel else float(l0.P))
        ones = np.ones((Oc, Cc, KH, KH), dtype=np.float32)
        e = (_conv_f64_im2col(eps, np.abs(w0), None, stride)[0]
             + _conv_f64_im2col(np.abs(a) + eps, ones, None, stride)[0] * sw0 / 2 + P0 / 2)
        a = c_ref[r].reshape(-1)
        eps = e.reshape(-1) + float(l1.s_a) / 2
        for i, (l, ql) in enumerate(zip(layers[1:], qp.layers[1:])):
            Wm = l.weight.astype(np.float64)
            e = np.abs(Wm) @ eps + (np.abs(a) + eps).sum() * float(ql.s_w) / 2 + float(ql.P) / 2
            pre = Wm @ a + (0 if l.bias is None else l.bias.astype(np.float64))
            if i == 0:
                a = np.maximum(pre, 0)
                eps = e + float(qp.layers[2].s_a) / 2
        assert np.all(np.abs(y_q[r].astype(np.float64) - y_fp[r]) <= e * (1 + 1e-6) + 1e-6), (r, y_q[r], y_fp[r], e)
    assert np.abs(y_q - y_fp).max() > 0


# ---- counter-based exploration noise: Philox-4x32-10 + Box-Muller ------------------------------------

def test_philox_known_answers():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_known_answers.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        c, k, want = [[int(w, 16) for w in part.split()] for part in line.split("|")]
        got = [int(v) for v in O.philox4x32_10(c, k)]
        assert got == want, (line, [hex(g) for g in got])
        n += 1
    assert n == 3
    # vectorised over counters: the same words as one counter at a time
    cs = np.array([[0, 1, 2, 3], [5, 0, 7, 0], [0xFFFFFFFF, 3, 0, 9]], dtype=np.uint64)
    many = O.philox4x32_10([cs[:, i] for i in range(4)], (11, 12))
    for r in range(3):
        one = O.philox4x32_10([int(v) for v in cs[r]], (11, 12))
        assert [int(m[r]) for m in many] == [int(v) for v in one]


def test_exploration_normals_are_standard_normal_and_keyed_by_row_column_seed():
    z = O.exploration_normals(1234, 0, 40000, 21)
    assert z.shape == (40000, 21) and np.isfinite(z).all()
    assert abs(z.mean()) < 4.0 / np.sqrt(z.size) and abs(z.var() - 1.0) < 0.01
    assert abs((z ** 3).mean()) < 0.02 and abs((z ** 4).mean() - 3.0) < 0.05               # skewness 0, kurtosis 3
    q = np.quantile(z, [0.001, 0.0228, 0.1587, 0.5, 0.8413, 0.9772, 0.999])
    assert np.allclose(q, [-3.0902, -2.0, -1.0, 0.0, 1.0, 2.0, 3.0902], atol=0.03)          # the normal quantiles
    assert np.abs(z).max() <= np.sqrt(-2.0 * np.log(0.5 * 2.0 ** -23)) + 1e-12             # largest radius the 23-bit uniform allows
    # neighbouring columns (cos / sin of one pair, the two pairs of one counter) and rows are uncorrelated
    for a, b in [(z[:, 0], z[:, 1]), (z[:, 0], z[:, 2]), (z[:, 3], z[:, 4]), (z[:-1, 5], z[1:, 5])]:
        assert abs(np.corrcoef(a, b)[0, 1]) < 0.02
    # a row's draws depend on (seed, absolute row, column) only: not on the batch or on how many columns are drawn
    assert np.array_equal(O.exploration_normals(1234, 100, 7, 21), z[100:107])
    assert np.array_equal(O.exploration_normals(1234, 0, 50, 6), z[:50, :6])
    assert not np.array_equal(O.exploration_normals(1235, 0, 50, 6), z[:50, :6])
    # rows beyond 2^32 use the second counter word
    hi = O.exploration_normals(9, 2 ** 32 + 5, 2, 4)
    assert not np.array_equal(hi, O.exploration_normals(9, 5, 2, 4))


def test_explore_seeded_is_explore_with_those_draws():
    rng = np.random.default_rng(5)
    y = np.tanh(rng.standard_normal((64, 6))).astype(np.float32)
    sigma = rng.uniform(0, 0.2, 64).astype(np.float32)
    got = O.explore_seeded(y, sigma, 77, row0=3)
    z = O.exploration_normals(77, 3, 64, 6).astype(np.float32)
    assert np.array_equal(got, O.explore(y, sigma, z))
    assert np.array_equal(O.explore_seeded(y, np.zeros(64, np.float32), 77), y)             # sigma 0: the policy's own action


# ---- the fp16 actor ------------------------------------------------------------------------------------

def _rne_binary16(fr: F) -> F:
    """correctly rounded binary16 (normal range) of an exact rational, independent of numpy's cast"""
    if fr == 0:
        return F(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = math.floor(math.log2(a))
    while F(2) ** e > a:
        e -= 1
    while F(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -14)                                   # subnormals share the smallest normal exponent
    ulp = F(2) ** (e - 10)
    return sign * _rne(a / ulp) * ulp


def test_fp16_cast_is_round_to_nearest_even():
    rng = np.random.default_rng(70)
    w = np.concatenate([rng.standard_normal(200) * 10.0 ** rng.uniform(-4, 3, 200),
                        [1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2049.0, 2051.0, 6.0e-8, 65504.0]]).astype(np.float32)   # ties and a subnormal
    got = O.cast_fp16(w)
    for x, g in zip(w.tolist(), got.tolist()):
        assert F(g) == _rne_binary16(F(x)), (x, g)
    rel = np.abs(got.astype(np.float64) - w.astype(np.float64)) / np.abs(w.astype(np.float64))
    assert rel[np.abs(w) > 1e-4].max() <= 2.0 ** -11


def test_fp16_forward_is_exact_on_a_power_of_two_grid():
    """Small integers times powers of two: every product and sum is exact in binary16 / 32 / 64, so the fp16
    forward must equal integer arithmetic exactly (a dropped bias, a transposed weight or a missing ReLU fails)."""
    rng = np.random.default_rng(71)
    w0 = rng.integers(-4, 5, (6, 5)).astype(np.float32) * 0.25
    b0 = rng.integers(-3, 4, 6).astype(np.float32) * 0.5
    w1 = rng.integers(-4, 5, (3, 6)).astype(np.float32) * 0.5
    obs = rng.integers(-8, 9, (11, 5)).astype(np.float32) * 0.125
    y, act, trace = O.forward_fp16([_L(w0, b0), _L(w1, None)], obs, "argmax")
    h = np.maximum(obs.astype(np.float64) @ w0.astype(np.float64).T + b0, 0.0)
    assert np.array_equal(trace[0].astype(np.float64), h)
    assert np.array_equal(y.astype(np.float64), h @ w1.astype(np.float64).T)
    assert np.array_equal(act, np.argmax(y, axis=1))


@pytest.mark.parametrize("dims,head", [([3, 4, 2], "tanh"), ([5, 16, 8, 3], "linear")])
def test_fp16_forward_close_to_fp_forward(dims, head):
    """|y16 - y| within the bound propagated from one binary16 rounding (relative 2^-11) per weight, input
    and hidden activation; and not vacuous: fp16 really differs from the un-rounded network."""
    rng = np.random.default_rng(72)
    layers = [_L((rng.standard_normal((dims[i + 1], dims[i])) * dims[i] ** -0.5).astype(np.float32),
                 (rng.standard_normal(dims[i + 1]) * 0.1).astype(np.float32)) for i in range(len(dims) - 1)]
    obs = rng.standard_normal((200, dims[0])).astype(np.float32)
    y16, _, _ = O.forward_fp16(layers, obs, head)
    y64, _ = O.forward_f64(layers, obs, head, "f32")
    u = 2.0 ** -11
    for r in range(obs.shape[0]):
        a = np.abs(obs[r].astype(np.float64))
        eps = a * u
        x = obs[r].astype(np.float64)
        for i, l in enumerate(layers):
            Wm = l.weight.astype(np.float64)
            e = np.abs(Wm) @ eps + (np.abs(Wm) * u) @ (np.abs(x) + eps)
            pre = Wm @ x + l.bias.astype(np.float64)
            if i + 1 < len(layers):
                x = np.maximum(pre, 0)
                eps = e + (np.abs(x) + e) * u
        assert np.all(np.abs(y16[r].astype(np.float64) - y64[r]) <= e * (1 + 1e-6) + 1e-7), (r, y16[r], y64[r], e)
    assert np.abs(y16 - y64).max() > 0
