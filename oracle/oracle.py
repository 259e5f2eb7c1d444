"""ctypes front end of the CPU checker (oracle/actorq_oracle.c) -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It never imports the CUDA package.  The C file holds every arithmetic
step; this file only sequences the steps layer by layer, in the order the paper's
actor runs them (quantize the broadcast policy once, then run int8 inference on
each observation), and keeps every intermediate so the tests can compare them.

Layer objects are duck-typed: .kind ("fc"/"conv"), .weight (float32 ndarray),
.bias (float32 ndarray or None), and for conv .stride and .in_hw.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "actorq_oracle.c")
_LIB = os.path.join(_HERE, "libactorq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc (strict IEEE float semantics, OpenMP over batch rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.actorq_ref_tensor_range.restype = C.c_int
        _lib.actorq_ref_layer_consts.restype = C.c_int
        _lib.actorq_ref_max_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def max_threads() -> int:
    return int(lib().actorq_ref_max_threads())


# ---- single steps ------------------------------------------------------------

def tensor_range(w: np.ndarray) -> Tuple[float, float, bool]:
    w = np.ascontiguousarray(w, dtype=np.float32)
    lo, hi = C.c_float(), C.c_float()
    bad = lib().actorq_ref_tensor_range(_p(w), C.c_longlong(w.size), C.byref(lo), C.byref(hi))
    return lo.value, hi.value, bool(bad)


def affine_params(rmin: float, rmax: float) -> Tuple[np.float32, int]:
    s, z = C.c_float(), C.c_int()
    lib().actorq_ref_affine_params(C.c_float(rmin), C.c_float(rmax), C.byref(s), C.byref(z))
    return np.float32(s.value), int(z.value)


def quantize_weights(w: np.ndarray) -> Tuple[np.ndarray, np.float32, int]:
    """Eq. 1-2 on one tensor: returns (codes, delta, zero_point)."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    lo, hi, bad = tensor_range(w)
    if bad:
        raise ValueError("non-finite weight")
    s, z = affine_params(lo, hi)
    q = np.empty(w.shape, dtype=np.int8)
    lib().actorq_ref_quantize_weights(_p(w), C.c_longlong(w.size), C.c_float(s), C.c_int(z), _p(q))
    return q, s, z


def dequantize(q: np.ndarray, s, z: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    out = np.empty(q.shape, dtype=np.float32)
    lib().actorq_ref_dequantize(_p(q), C.c_longlong(q.size), C.c_float(s), C.c_int(z), _p(out))
    return out


def quantize_input_f32(x: np.ndarray, s_a, z_a: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.int8)
    lib().actorq_ref_quantize_input_f32(_p(x), C.c_longlong(x.size), C.c_float(s_a), C.c_int(z_a), _p(q))
    return q


def quantize_input_u8(u: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(u, dtype=np.uint8)
    q = np.empty(u.shape, dtype=np.int8)
    lib().actorq_ref_quantize_input_u8(_p(u), C.c_longlong(u.size), _p(q))
    return q


def layer_consts(s_a, s_w, s_out, bias: Optional[np.ndarray], n_out: int):
    P, M = C.c_float(), C.c_float()
    bq = np.zeros(n_out, dtype=np.int32)
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    bad = lib().actorq_ref_layer_consts(C.c_float(s_a), C.c_float(s_w), C.c_float(s_out), _p(b),
                                        C.c_int(n_out), C.byref(P), C.byref(M), _p(bq))
    if bad:
        raise ValueError("non-finite bias")
    return np.float32(P.value), np.float32(M.value), bq


def fc_acc(a: np.ndarray, z_a: int, w_q: np.ndarray, z_w: int, bias_q: Optional[np.ndarray],
           expanded: bool = False) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int8)
    w_q = np.ascontiguousarray(w_q, dtype=np.int8)
    B, K = a.shape
    N = w_q.shape[0]
    assert w_q.shape[1] == K and K <= 16384
    acc = np.empty((B, N), dtype=np.int32)
    fn = lib().actorq_ref_fc_acc_expanded if expanded else lib().actorq_ref_fc_acc
    fn(_p(a), C.c_longlong(B), C.c_int(K), C.c_int(z_a), _p(w_q), C.c_int(N), C.c_int(z_w), _p(bias_q), _p(acc))
    return acc


def conv_acc(a: np.ndarray, z_a: int, w_q: np.ndarray, stride: int, z_w: int,
             bias_q: Optional[np.ndarray]) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int8)
    w_q = np.ascontiguousarray(w_q, dtype=np.int8)
    B, Cc, H, W = a.shape
    O, C2, KH, KW = w_q.shape
    assert C2 == Cc
    OH, OW = (H - KH) // stride + 1, (W - KW) // stride + 1
    acc = np.empty((B, O, OH, OW), dtype=np.int32)
    lib().actorq_ref_conv_acc(_p(a), C.c_longlong(B), C.c_int(Cc), C.c_int(H), C.c_int(W), C.c_int(z_a),
                              _p(w_q), C.c_int(O), C.c_int(KH), C.c_int(KW), C.c_int(stride), C.c_int(z_w),
                              _p(bias_q), _p(acc))
    return acc


def requantize_relu(acc: np.ndarray, M, z_out: int) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    q = np.empty(acc.shape, dtype=np.int8)
    lib().actorq_ref_requantize_relu(_p(acc), C.c_longlong(acc.size), C.c_float(M), C.c_int(z_out), _p(q))
    return q


def head_dequant(acc: np.ndarray, P, tanh: bool) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    y = np.empty(acc.shape, dtype=np.float32)
    lib().actorq_ref_head_dequant(_p(acc), C.c_longlong(acc.size), C.c_float(P), C.c_int(int(tanh)), _p(y))
    return y


def explore(y: np.ndarray, sigma: np.ndarray, noise: np.ndarray) -> np.ndarray:
    """Actor exploration (Section 5, set-up: Gaussian noise layer on the policy output, sigma per
    actor): clip(y + sigma[row] * noise, -1, 1), one binary32 multiply and one binary32 add.
    Reading: the paper does not mention the clip; actions of a tanh policy live in [-1, 1]."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    t = (np.asarray(sigma, dtype=np.float32).reshape(-1, 1) * np.asarray(noise, dtype=np.float32)).astype(np.float32)
    v = (y + t).astype(np.float32)
    return np.minimum(np.maximum(v, np.float32(-1.0)), np.float32(1.0)).astype(np.float32)


def argmax(y: np.ndarray) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float32)
    B, N = y.shape
    act = np.empty(B, dtype=np.int32)
    lib().actorq_ref_argmax(_p(y), C.c_longlong(B), C.c_int(N), _p(act))
    return act


# ---- whole policy --------------------------------------------------------------

# ---- per-output-channel variants (Section 3.2: per-channel quantization of conv layers) -----

def quantize_weights_per_channel(w: np.ndarray):
    """Eq. 1-2 applied to each output channel (row w[n]) on its own: codes, s_w[N], z_w[N]."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    N = w.shape[0]
    q = np.empty(w.shape, dtype=np.int8)
    s = np.empty(N, dtype=np.float32)
    z = np.empty(N, dtype=np.int32)
    for n in range(N):
        q[n], s[n], z[n] = quantize_weights(w[n])
    return q, s, z


def layer_consts_per_channel(s_a, s_w: np.ndarray, s_out, bias: Optional[np.ndarray]):
    """P[n] = s_a * s_w[n], M[n] = P[n] / s_out, bias_q[n] = rne(b[n] / P[n]), channel by channel."""
    N = len(s_w)
    P = np.empty(N, dtype=np.float32)
    M = np.empty(N, dtype=np.float32)
    bias_q = np.zeros(N, dtype=np.int32)
    for n in range(N):
        b = None if bias is None else np.ascontiguousarray(bias[n:n + 1], dtype=np.float32)
        P[n], M[n], bq = layer_consts(s_a, s_w[n], s_out, b, 1)
        bias_q[n] = bq[0]
    return P, M, bias_q


def fc_acc_pc(a: np.ndarray, z_a: int, w_q: np.ndarray, z_w: np.ndarray, bias_q: Optional[np.ndarray]) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int8)
    w_q = np.ascontiguousarray(w_q, dtype=np.int8)
    z_w = np.ascontiguousarray(z_w, dtype=np.int32)
    B, K = a.shape
    N = w_q.shape[0]
    acc = np.empty((B, N), dtype=np.int32)
    bq = None if bias_q is None else np.ascontiguousarray(bias_q, dtype=np.int32)
    lib().actorq_ref_fc_acc_pc(_p(a), C.c_longlong(B), C.c_int(K), C.c_int(int(z_a)), _p(w_q), C.c_int(N), _p(z_w), _p(bq), _p(acc))
    return acc


def conv_acc_pc(a: np.ndarray, z_a: int, w_q: np.ndarray, stride: int, z_w: np.ndarray,
                bias_q: Optional[np.ndarray]) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int8)
    w_q = np.ascontiguousarray(w_q, dtype=np.int8)
    z_w = np.ascontiguousarray(z_w, dtype=np.int32)
    B, Cc, H, W = a.shape
    O, _, KH, KW = w_q.shape
    OH, OW = (H - KH) // stride + 1, (W - KW) // stride + 1
    acc = np.empty((B, O, OH, OW), dtype=np.int32)
    bq = None if bias_q is None else np.ascontiguousarray(bias_q, dtype=np.int32)
    lib().actorq_ref_conv_acc_pc(_p(a), C.c_longlong(B), C.c_int(Cc), C.c_int(H), C.c_int(W), C.c_int(int(z_a)), _p(w_q),
                                 C.c_int(O), C.c_int(KH), C.c_int(KW), C.c_int(stride), _p(z_w), _p(bq), _p(acc))
    return acc


def requantize_relu_pc(acc: np.ndarray, M: np.ndarray, z_out: int) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    M = np.ascontiguousarray(M, dtype=np.float32)
    B, N = acc.shape[0], acc.shape[1]
    inner = int(np.prod(acc.shape[2:])) if acc.ndim > 2 else 1
    q = np.empty(acc.shape, dtype=np.int8)
    lib().actorq_ref_requantize_relu_pc(_p(acc), C.c_longlong(B), C.c_int(N), C.c_longlong(inner), _p(M), C.c_int(int(z_out)), _p(q))
    return q


def head_dequant_pc(acc: np.ndarray, P: np.ndarray, tanh: bool) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    P = np.ascontiguousarray(P, dtype=np.float32)
    B, N = acc.shape
    y = np.empty((B, N), dtype=np.float32)
    lib().actorq_ref_head_dequant_pc(_p(acc), C.c_longlong(B), C.c_int(N), _p(P), C.c_int(int(tanh)), _p(y))
    return y


@dataclass
class QLayer:
    kind: str
    w_q: np.ndarray
    s_w: np.float32
    z_w: int
    s_a: np.float32
    z_a: int
    P: np.float32
    M: np.float32          # meaningful for hidden layers only
    z_out: int             # next layer's activation zero-point (hidden layers only)
    bias_q: np.ndarray
    stride: int = 1
    in_hw: Tuple[int, int] = (0, 0)
    per_channel: bool = False      # s_w, z_w, P, M are then arrays over the output channels


@dataclass
class QPolicy:
    layers: List[QLayer]
    head: str
    obs_dtype: str


def quantize_policy(layers: Sequence, input_ranges: Sequence[Tuple[float, float]], head: str,
                    obs_dtype: str) -> QPolicy:
    """The quantizer block: every weight tensor through Eq. 1-2, plus the per-layer constants."""
    n = len(layers)
    act = []
    for i in range(n):
        if i == 0 and obs_dtype == "u8":
            act.append((np.float32(1.0) / np.float32(255.0), -128))
        else:
            act.append(affine_params(*input_ranges[i]))
    out = []
    for i, l in enumerate(layers):
        s_a, z_a = act[i]
        s_out, z_out = act[i + 1] if i + 1 < n else (np.float32(1.0), 0)
        n_out = l.weight.shape[0]
        pc = bool(getattr(l, "per_channel", False))
        if pc:
            w_q, s_w, z_w = quantize_weights_per_channel(l.weight)
            P, M, bias_q = layer_consts_per_channel(s_a, s_w, s_out, l.bias)
        else:
            w_q, s_w, z_w = quantize_weights(l.weight)
            P, M, bias_q = layer_consts(s_a, s_w, s_out, l.bias, n_out)
        out.append(QLayer(l.kind, w_q, s_w, z_w, s_a, z_a, P, M, z_out, bias_q,
                          getattr(l, "stride", 1), tuple(getattr(l, "in_hw", (0, 0))), pc))
    return QPolicy(out, head, obs_dtype)


def forward(qp: QPolicy, obs: np.ndarray):
    """int8 inference of the quantized policy.  Returns (out fp32 [B][out_dim], actions or None,
    trace) where trace[i] = (acc int32, act_q int8 or None) for layer i in [batch][...] order
    (conv layers in [B][C][H][W] order, i.e. flattened (c, h, w))."""
    l0 = qp.layers[0]
    if qp.obs_dtype == "u8":
        a = quantize_input_u8(obs)
    else:
        a = quantize_input_f32(obs, l0.s_a, l0.z_a)
    trace = []
    n = len(qp.layers)
    for i, l in enumerate(qp.layers):
        if l.kind == "conv":
            acc = (conv_acc_pc if l.per_channel else conv_acc)(a, l.z_a, l.w_q, l.stride, l.z_w, l.bias_q)
        else:
            acc = (fc_acc_pc if l.per_channel else fc_acc)(a.reshape(a.shape[0], -1), l.z_a, l.w_q, l.z_w, l.bias_q)
        if i + 1 < n:
            a = (requantize_relu_pc if l.per_channel else requantize_relu)(acc, l.M, l.z_out)
            trace.append((acc, a))
        else:
            trace.append((acc, None))
            y = (head_dequant_pc if l.per_channel else head_dequant)(acc, l.P, qp.head == "tanh")
    actions = argmax(y) if qp.head == "argmax" else None
    return y, actions, trace


def forward_f64(layers: Sequence, obs: np.ndarray, head: str, obs_dtype: str):
    """The un-quantized network in double precision; returns (y, per-layer inputs)."""
    x = obs.astype(np.float64)
    if obs_dtype == "u8":
        x = x / 255.0
    inputs = []
    n = len(layers)
    for i, l in enumerate(layers):
        inputs.append(x)
        relu = int(i + 1 < n)
        w = np.ascontiguousarray(l.weight, dtype=np.float32)
        b = None if l.bias is None else np.ascontiguousarray(l.bias, dtype=np.float32)
        if l.kind == "conv":
            x = np.ascontiguousarray(x)
            B, Cc, H, W = x.shape
            O, _, KH, KW = w.shape
            OH, OW = (H - KH) // l.stride + 1, (W - KW) // l.stride + 1
            y = np.empty((B, O, OH, OW), dtype=np.float64)
            lib().actorq_ref_conv_f64(_p(x), C.c_longlong(B), C.c_int(Cc), C.c_int(H), C.c_int(W), _p(w), _p(b),
                                      C.c_int(O), C.c_int(KH), C.c_int(KW), C.c_int(l.stride), C.c_int(relu), _p(y))
        else:
            x = np.ascontiguousarray(x.reshape(x.shape[0], -1))
            B, K = x.shape
            N = w.shape[0]
            y = np.empty((B, N), dtype=np.float64)
            lib().actorq_ref_fc_f64(_p(x), C.c_longlong(B), C.c_int(K), _p(w), _p(b), C.c_int(N), C.c_int(relu), _p(y))
        x = y
    if head == "tanh":
        x = np.tanh(x)
    return x, inputs


# ---- counter-based exploration noise (Section 5, set-up: Gaussian noise on the actor's policy output) ------
# The paper does not say how the actor draws its noise.  Reading taken here: row b, column n of a forward
# call with seed s gets the standard normal z[b][n] of a counter-based generator, so that a row's noise does
# not depend on the batch it travels in:
#   (x0, x1, x2, x3) = Philox-4x32-10(counter = (b mod 2^32, b div 2^32, n div 4, 0), key = (s mod 2^32, s div 2^32))
#   the pair (x0, x1) serves columns 4j, 4j + 1 and (x2, x3) columns 4j + 2, 4j + 3 of block j = n div 4:
#   u1 = ((xa >> 9) + 1/2) 2^-23, u2 = ((xb >> 9) + 1/2) 2^-23            (24 significant bits: exact in binary32)
#   z_even = sqrt(-2 ln u1) cos(2 pi u2),  z_odd = sqrt(-2 ln u1) sin(2 pi u2)       (Box-Muller)
# Philox-4x32-10 is the generator of Salmon, Moraes, Dror and Shaw, "Parallel random numbers: as easy as
# 1, 2, 3" (SC'11), written out below from its definition; the checker evaluates the transform in double.

_PHILOX_M0, _PHILOX_M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_PHILOX_W0, _PHILOX_W1 = np.uint64(0x9E3779B9), np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """counter: 4 arrays (or ints) of 32-bit words, key: 2 words; returns 4 uint64 arrays holding 32-bit words."""
    c = [np.asarray(x, dtype=np.uint64) & _MASK32 for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = (np.uint64(int(key[0]) & 0xFFFFFFFF), np.uint64(int(key[1]) & 0xFFFFFFFF))
    for _ in range(10):
        p0 = _PHILOX_M0 * c[0]                 # 32 x 32 -> 64-bit products
        p1 = _PHILOX_M1 * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c = [hi1 ^ c[1] ^ k0, lo1, hi0 ^ c[3] ^ k1, lo0]
        k0 = (k0 + _PHILOX_W0) & _MASK32       # the key schedule: one Weyl step per round
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return c


def exploration_normals(seed: int, row0: int, rows: int, cols: int) -> np.ndarray:
    """z[b][n] (float64) for rows row0 .. row0 + rows - 1 and columns 0 .. cols - 1 of a call with this seed."""
    b = (np.arange(rows, dtype=np.uint64) + np.uint64(row0)).reshape(-1, 1)
    n = np.arange(cols, dtype=np.uint64).reshape(1, -1)
    x = philox4x32_10((b & _MASK32, b >> np.uint64(32), n >> np.uint64(2), np.uint64(0)), (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    second_pair = ((n >> np.uint64(1)) & np.uint64(1)) == 1
    xa = np.where(second_pair, x[2], x[0])
    xb = np.where(second_pair, x[3], x[1])
    u1 = ((xa >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23
    u2 = ((xb >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23
    radius = np.sqrt(-2.0 * np.log(u1))
    odd = (n & np.uint64(1)) == 1
    return np.where(odd, radius * np.sin(2.0 * np.pi * u2), radius * np.cos(2.0 * np.pi * u2))


def explore_seeded(y: np.ndarray, sigma: np.ndarray, seed: int, row0: int = 0) -> np.ndarray:
    """explore() with the draws of exploration_normals, rounded to binary32 before the multiply."""
    z = exploration_normals(seed, row0, y.shape[0], y.shape[1]).astype(np.float32)
    return explore(y, sigma, z)


# ---- the fp16 actor (Section 3.2: policies are quantized "to fp16 and int8"; the q = 16 rows of the
# communication-vs-computation study) ---------------------------------------------------------------
# Reading (the paper names the precision, not the arithmetic): weights and observations are rounded to
# binary16 (round to nearest even); a layer is y[n] = sum_k a[k] w[n][k] + b[n] with the bias kept in
# binary32; hidden layers apply ReLU and round the result to binary16 for the next layer; the head
# applies tanh (or nothing).  A product of two binary16 numbers is exact in binary32 and in binary64,
# so the checker forms the sum in binary64 (exact to ~1e-16 relative of the sum of magnitudes) and rounds
# ONCE; an implementation that accumulates in binary32 differs by its accumulation error and, where that
# moves a value across a rounding boundary, by one binary16 step (see the tolerance in the parity test).

def cast_fp16(w: np.ndarray) -> np.ndarray:
    """round to nearest even binary16 (values beyond 65504 become +-inf, as the format prescribes)"""
    return np.asarray(w, dtype=np.float32).astype(np.float16)


def forward_fp16(layers: Sequence, obs: np.ndarray, head: str):
    """Returns (out float32 [B][out_dim], actions or None, trace) with trace[i] = layer i's binary16 output
    activations (hidden layers) or its binary32 pre-activation (last layer)."""
    a = cast_fp16(obs).astype(np.float64)
    trace = []
    n = len(layers)
    y = None
    for i, l in enumerate(layers):
        w16 = cast_fp16(l.weight).astype(np.float64)
        acc = a.reshape(a.shape[0], -1) @ w16.T
        if l.bias is not None:
            acc = acc + np.asarray(l.bias, dtype=np.float32).astype(np.float64)
        if i + 1 < n:
            h = np.maximum(acc, 0.0).astype(np.float16)          # one rounding of the (to 1e-16) exact value
            trace.append(h)
            a = h.astype(np.float64)
        else:
            pre = acc.astype(np.float32)
            trace.append(pre)
            y = np.tanh(acc).astype(np.float32) if head == "tanh" else pre
    actions = argmax(y) if head == "argmax" else None
    return y, actions, trace
