"""Thin ctypes binding of libactorq.so: argument marshalling only.

Function names mirror the C ABI (include/actorq.h).  torch supplies device memory and the
current stream; every arithmetic step runs inside the CUDA library.  Importing this module
without the built library, or calling it without a CUDA device, raises -- there is no
fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libactorq.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NONFINITE, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT, ERR_SCRATCH_LIMIT = range(8)
FC, CONV2D = 0, 1
HEAD = {"tanh": 0, "argmax": 1, "linear": 2}
OBS = {"f32": 0, "u8": 1}
STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "NONFINITE", "NOMEM", "CUDA", "TIMEOUT", "SCRATCH_LIMIT"]
NOALLOC_SCRATCH_BYTES = 64 << 20

EXPORTS = ["actorq_policy_blob_bytes", "actorq_policy_export_blob", "actorq_policy_import_blob", "actorq_quantize_params", "actorq_policy_forward", "actorq_policy_forward_noalloc", "actorq_free", "actorq_policy_export_layer",
           "actorq_policy_forward_debug", "actorq_policy_last_device_status",
           "actorq_policy_last_launch_count", "actorq_policy_timeout_info", "actorq_selftest_bounded_wait", "actorq_selftest_int8_mma_peak",
           "actorq_policy_set_fused_variant", "actorq_policy_forward_host", "actorq_policy_export_layer_channels", "actorq_policy_forward_explore", "actorq_policy_forward_explore_seeded", "actorq_cast_params_fp16", "actorq_version"]


class LayerDesc(C.Structure):
    _fields_ = [("kind", C.c_int), ("in_features", C.c_int), ("out_features", C.c_int),
                ("in_c", C.c_int), ("in_h", C.c_int), ("in_w", C.c_int), ("out_c", C.c_int),
                ("kh", C.c_int), ("kw", C.c_int), ("stride", C.c_int),
                ("weight", C.c_void_p), ("bias", C.c_void_p), ("per_channel", C.c_int)]


class Range(C.Structure):
    _fields_ = [("min", C.c_float), ("max", C.c_float)]


class ActorQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where} failed: ACTORQ_ERR_{name}")


_lib = None


def load() -> C.CDLL:
    """Load the in-tree CUDA library (build it first with paper_1910_01055_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_1910_01055_b200.build`")
        lib = C.CDLL(LIB_PATH)
        lib.actorq_quantize_params.argtypes = [C.POINTER(LayerDesc), C.c_int, C.POINTER(Range), C.c_int, C.c_int,
                                               C.c_void_p, C.POINTER(C.c_void_p)]
        lib.actorq_policy_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.actorq_policy_forward_noalloc.argtypes = lib.actorq_policy_forward.argtypes
        lib.actorq_free.argtypes = [C.c_void_p]
        lib.actorq_free.restype = None
        lib.actorq_policy_export_layer.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(C.c_float),
                                                   C.POINTER(C.c_int), C.c_void_p]
        lib.actorq_policy_forward_debug.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p,
                                                    C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.actorq_policy_last_device_status.argtypes = [C.c_void_p]
        lib.actorq_policy_last_launch_count.argtypes = [C.c_void_p]
        lib.actorq_version.restype = C.c_char_p
        _lib = lib
    return _lib


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _check(code: int, where: str) -> None:
    if code != OK:
        raise ActorQError(code, where)


def make_layer_descs(layers: Sequence[dict]) -> "C.Array[LayerDesc]":
    """layers: dicts with 'weight' (cuda float32 tensor, FC [out][in] or conv [O][I][KH][KW]),
    optional 'bias', and for conv 'stride', 'in_hw'."""
    arr = (LayerDesc * len(layers))()
    for d, l in zip(arr, layers):
        w = l["weight"]
        assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
        b = l.get("bias")
        if b is not None:
            assert b.is_cuda and b.dtype == torch.float32 and b.is_contiguous()
        d.per_channel = 1 if l.get("per_channel") else 0
        d.weight = w.data_ptr()
        d.bias = b.data_ptr() if b is not None else None
        if w.dim() == 2:
            d.kind, d.out_features, d.in_features = FC, w.shape[0], w.shape[1]
        else:
            d.kind = CONV2D
            d.out_c, d.in_c, d.kh, d.kw = w.shape
            d.in_h, d.in_w = l["in_hw"]
            d.stride = l.get("stride", 1)
    return arr


def actorq_quantize_params(layers: Sequence[dict], input_ranges: Sequence[Tuple[float, float]], head: str,
                           obs_dtype: str, policy: Optional[C.c_void_p] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> C.c_void_p:
    """Quantize (policy=None: create) or re-quantize in place; returns the policy handle."""
    lib = load()
    descs = make_layer_descs(layers)
    ranges = (Range * len(layers))(*[Range(float(a), float(b)) for a, b in input_ranges])
    handle = policy if policy is not None else C.c_void_p(None)
    rc = lib.actorq_quantize_params(descs, len(layers), ranges, HEAD[head], OBS[obs_dtype], _stream_ptr(stream),
                                    C.byref(handle))
    _check(rc, "actorq_quantize_params")
    return handle


def actorq_policy_forward(policy: C.c_void_p, obs: torch.Tensor, out: torch.Tensor,
                          actions: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    lib = load()
    assert obs.is_cuda and obs.is_contiguous() and out.is_cuda and out.is_contiguous() and out.dtype == torch.float32
    if actions is not None:
        assert actions.is_cuda and actions.dtype == torch.int32 and actions.is_contiguous()
    rc = lib.actorq_policy_forward(policy, obs.data_ptr(), obs.shape[0], out.data_ptr(),
                                   actions.data_ptr() if actions is not None else None, _stream_ptr(stream))
    _check(rc, "actorq_policy_forward")


def actorq_cast_params_fp16(layers: Sequence[dict], head: str, obs_dtype: str, policy: Optional[C.c_void_p] = None,
                            stream: Optional[torch.cuda.Stream] = None) -> C.c_void_p:
    """Cast the fp32 policy to binary16 (the paper's q = 16 actor); returns the (new or re-cast) policy handle."""
    lib = load()
    n = len(layers)
    descs = (LayerDesc * n)()
    for i, l in enumerate(layers):
        w = l["weight"]
        assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
        assert w.dim() == 2, "the fp16 actor takes fully connected layers"
        b = l.get("bias")
        descs[i].kind = FC
        descs[i].out_features, descs[i].in_features = w.shape
        descs[i].weight = w.data_ptr()
        descs[i].bias = b.data_ptr() if b is not None else None
    handle = policy if policy is not None else C.c_void_p(None)
    lib.actorq_cast_params_fp16.argtypes = [C.POINTER(LayerDesc), C.c_int, C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_void_p)]
    _check(lib.actorq_cast_params_fp16(descs, n, HEAD[head], OBS[obs_dtype], _stream_ptr(stream), C.byref(handle)), "actorq_cast_params_fp16")
    return handle


def actorq_policy_forward_explore(policy: C.c_void_p, obs: torch.Tensor, sigma: torch.Tensor, noise: torch.Tensor,
                                  out: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """tanh policies: out = clamp(tanh(y) + sigma[row] * noise, -1, 1); sigma [B], noise [B][out_dim] (cuda float32)."""
    lib = load()
    for t in (obs, sigma, noise, out):
        assert t.is_cuda and t.is_contiguous()
    assert sigma.dtype == torch.float32 and noise.dtype == torch.float32 and out.dtype == torch.float32
    assert sigma.shape[0] == obs.shape[0] and noise.shape == out.shape
    lib.actorq_policy_forward_explore.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    rc = lib.actorq_policy_forward_explore(policy, obs.data_ptr(), obs.shape[0], sigma.data_ptr(), noise.data_ptr(),
                                           out.data_ptr(), _stream_ptr(stream))
    _check(rc, "actorq_policy_forward_explore")


def actorq_policy_forward_explore_seeded(policy: C.c_void_p, obs: torch.Tensor, sigma: torch.Tensor, seed: int, out: torch.Tensor,
                                         first_row: int = 0, stream: Optional[torch.cuda.Stream] = None) -> None:
    """tanh policies: out = clamp(tanh(y) + sigma[row] * z, -1, 1) with z drawn by the library's counter-based
    generator from (seed, first_row + row, column); see actorq.h."""
    lib = load()
    for t in (obs, sigma, out):
        assert t.is_cuda and t.is_contiguous()
    assert sigma.dtype == torch.float32 and out.dtype == torch.float32 and sigma.shape[0] == obs.shape[0]
    lib.actorq_policy_forward_explore_seeded.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p, C.c_ulonglong,
                                                         C.c_longlong, C.c_void_p, C.c_void_p]
    rc = lib.actorq_policy_forward_explore_seeded(policy, obs.data_ptr(), obs.shape[0], sigma.data_ptr(), seed, first_row,
                                                  out.data_ptr(), _stream_ptr(stream))
    _check(rc, "actorq_policy_forward_explore_seeded")


def actorq_policy_forward_host(policy: C.c_void_p, obs: torch.Tensor, out: torch.Tensor,
                               actions: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None) -> None:
    """Forward with HOST tensors (pin them for the copies to overlap the compute): chunked, pipelined
    copies in / forward / copies out; complete when `stream` has reached the end of the call."""
    lib = load()
    assert not obs.is_cuda and obs.is_contiguous() and not out.is_cuda and out.is_contiguous() and out.dtype == torch.float32
    if actions is not None:
        assert not actions.is_cuda and actions.dtype == torch.int32 and actions.is_contiguous()
    lib.actorq_policy_forward_host.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p, C.c_void_p]
    rc = lib.actorq_policy_forward_host(policy, obs.data_ptr(), obs.shape[0], out.data_ptr(),
                                        actions.data_ptr() if actions is not None else None, _stream_ptr(stream))
    _check(rc, "actorq_policy_forward_host")


def actorq_policy_forward_noalloc(policy: C.c_void_p, obs: torch.Tensor, out: torch.Tensor,
                                  actions: Optional[torch.Tensor] = None,
                                  stream: Optional[torch.cuda.Stream] = None) -> None:
    """Forward for callers that must not allocate device memory: same results as
    actorq_policy_forward, activations kept in the library's fixed scratch array (batch limited,
    ActorQError with ERR_SCRATCH_LIMIT beyond it; calls that overlap on the GPU race)."""
    lib = load()
    assert obs.is_cuda and obs.is_contiguous() and out.is_cuda and out.is_contiguous() and out.dtype == torch.float32
    if actions is not None:
        assert actions.is_cuda and actions.dtype == torch.int32 and actions.is_contiguous()
    rc = lib.actorq_policy_forward_noalloc(policy, obs.data_ptr(), obs.shape[0], out.data_ptr(),
                                           actions.data_ptr() if actions is not None else None, _stream_ptr(stream))
    _check(rc, "actorq_policy_forward_noalloc")


def actorq_policy_forward_debug(policy: C.c_void_p, obs: torch.Tensor, out: torch.Tensor,
                                actions: Optional[torch.Tensor], layer: int, acc: torch.Tensor,
                                act_q: Optional[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
    lib = load()
    assert acc.is_cuda and acc.dtype == torch.int32 and acc.is_contiguous()
    if act_q is not None:
        assert act_q.is_cuda and act_q.dtype == torch.int8 and act_q.is_contiguous()
    rc = lib.actorq_policy_forward_debug(policy, obs.data_ptr(), obs.shape[0], out.data_ptr(),
                                         actions.data_ptr() if actions is not None else None, layer,
                                         acc.data_ptr(), act_q.data_ptr() if act_q is not None else None,
                                         _stream_ptr(stream))
    _check(rc, "actorq_policy_forward_debug")


def actorq_policy_export_layer(policy: C.c_void_p, layer: int, w_q: torch.Tensor,
                               stream: Optional[torch.cuda.Stream] = None) -> Tuple[float, int]:
    lib = load()
    assert w_q.is_cuda and w_q.dtype == torch.int8 and w_q.is_contiguous()
    s, z = C.c_float(), C.c_int()
    rc = lib.actorq_policy_export_layer(policy, layer, w_q.data_ptr(), C.byref(s), C.byref(z), _stream_ptr(stream))
    _check(rc, "actorq_policy_export_layer")
    return s.value, z.value


def actorq_policy_export_layer_channels(policy: C.c_void_p, layer: int, w_q: torch.Tensor,
                                        stream: Optional[torch.cuda.Stream] = None):
    """Codes (into w_q), per-channel deltas and zero-points of a layer quantized per output channel."""
    import numpy as np
    lib = load()
    assert w_q.is_cuda and w_q.dtype == torch.int8 and w_q.is_contiguous()
    n = w_q.shape[0]
    s = np.empty(n, dtype=np.float32)
    z = np.empty(n, dtype=np.int32)
    lib.actorq_policy_export_layer_channels.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    rc = lib.actorq_policy_export_layer_channels(policy, layer, w_q.data_ptr(), s.ctypes.data, z.ctypes.data, _stream_ptr(stream))
    _check(rc, "actorq_policy_export_layer_channels")
    return s, z


def actorq_policy_last_device_status(policy: C.c_void_p) -> int:
    return int(load().actorq_policy_last_device_status(policy))


def actorq_policy_timeout_info(policy: C.c_void_p) -> dict:
    """Where the first timed-out device wait gave up (after a TIMEOUT status); clears the report."""
    info = (C.c_int * 8)()
    lib = load()
    lib.actorq_policy_timeout_info.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    _check(lib.actorq_policy_timeout_info(policy, info), "actorq_policy_timeout_info")
    return {"reported": bool(info[0]), "block": info[1], "warp": info[2], "barrier_offset": info[3], "parity": info[4]}


def actorq_policy_blob_bytes(policy: C.c_void_p) -> int:
    lib = load()
    n = C.c_longlong()
    lib.actorq_policy_blob_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_longlong)]
    _check(lib.actorq_policy_blob_bytes(policy, C.byref(n)), "actorq_policy_blob_bytes")
    return int(n.value)


def actorq_policy_export_blob(policy: C.c_void_p, blob: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Write the quantized policy into `blob` (cuda uint8 tensor of at least blob_bytes)."""
    lib = load()
    assert blob.is_cuda and blob.dtype == torch.uint8 and blob.is_contiguous()
    lib.actorq_policy_export_blob.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p]
    _check(lib.actorq_policy_export_blob(policy, blob.data_ptr(), blob.numel(), _stream_ptr(stream)), "actorq_policy_export_blob")


def actorq_policy_import_blob(policy: C.c_void_p, blob: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Load a blob written by a policy of the same architecture into `policy`."""
    lib = load()
    assert blob.is_cuda and blob.dtype == torch.uint8 and blob.is_contiguous()
    lib.actorq_policy_import_blob.argtypes = [C.c_void_p, C.c_void_p, C.c_longlong, C.c_void_p]
    _check(lib.actorq_policy_import_blob(policy, blob.data_ptr(), blob.numel(), _stream_ptr(stream)), "actorq_policy_import_blob")


def actorq_selftest_bounded_wait(policy: C.c_void_p, limit_ns: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launch the never-satisfied bounded wait (see actorq.h); read the status afterwards."""
    lib = load()
    lib.actorq_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_longlong, C.c_void_p]
    _check(lib.actorq_selftest_bounded_wait(policy, limit_ns, _stream_ptr(stream)), "actorq_selftest_bounded_wait")


def actorq_selftest_int8_mma_peak(policy: C.c_void_p, mma_groups: int, a_in_tmem: bool = False,
                                  stream: Optional[torch.cuda.Stream] = None) -> int:
    """Launch the bare int8 MMA loop (see actorq.h); returns the integer operations of the launch."""
    lib = load()
    lib.actorq_selftest_int8_mma_peak.argtypes = [C.c_void_p, C.c_longlong, C.c_int, C.POINTER(C.c_longlong), C.c_void_p]
    ops = C.c_longlong(0)
    _check(lib.actorq_selftest_int8_mma_peak(policy, mma_groups, int(a_in_tmem), C.byref(ops), _stream_ptr(stream)),
           "actorq_selftest_int8_mma_peak")
    return int(ops.value)


def actorq_policy_set_fused_variant(policy: C.c_void_p, variant: int) -> None:
    """0: library picks, 1: single-CTA fused MLP kernel, 2: CTA-pair kernel, 3: layer at a time, 4: resident weights (see actorq.h)."""
    lib = load()
    lib.actorq_policy_set_fused_variant.argtypes = [C.c_void_p, C.c_int]
    _check(lib.actorq_policy_set_fused_variant(policy, variant), "actorq_policy_set_fused_variant")


def actorq_policy_last_launch_count(policy: C.c_void_p) -> int:
    return int(load().actorq_policy_last_launch_count(policy))


def actorq_free(policy: Optional[C.c_void_p]) -> None:
    if policy is not None and policy.value:
        load().actorq_free(policy)
        policy.value = None


def actorq_version() -> str:
    return load().actorq_version().decode()


class QuantizedPolicy:
    """Convenience owner of one policy handle: quantize(), forward(), close()."""

    def __init__(self, head: str, obs_dtype: str):
        if not torch.cuda.is_available():
            raise RuntimeError("actorq needs a CUDA device; there is no CPU path")
        load()
        self.head, self.obs_dtype = head, obs_dtype
        self.handle: Optional[C.c_void_p] = None
        self.out_dim = None
        self._keep = None

    def quantize(self, layers: Sequence[dict], input_ranges, stream=None) -> "QuantizedPolicy":
        self.handle = actorq_quantize_params(layers, input_ranges, self.head, self.obs_dtype, self.handle, stream)
        w = layers[-1]["weight"]
        self.out_dim = w.shape[0]
        return self

    def forward(self, obs: torch.Tensor, out: Optional[torch.Tensor] = None,
                actions: Optional[torch.Tensor] = None, stream=None):
        B = obs.shape[0]
        if out is None:
            out = torch.empty((B, self.out_dim), dtype=torch.float32, device=obs.device)
        if self.head == "argmax" and actions is None:
            actions = torch.empty((B,), dtype=torch.int32, device=obs.device)
        actorq_policy_forward(self.handle, obs, out, actions, stream)
        return out, actions

    def status(self) -> int:
        return actorq_policy_last_device_status(self.handle)

    def close(self) -> None:
        actorq_free(self.handle)
        self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Fp16Policy(QuantizedPolicy):
    """The same owner for a policy cast to binary16 (actorq_cast_params_fp16): quantize() casts."""

    def quantize(self, layers: Sequence[dict], input_ranges=None, stream=None) -> "Fp16Policy":
        self.handle = actorq_cast_params_fp16(layers, self.head, self.obs_dtype, self.handle, stream)
        self.out_dim = layers[-1]["weight"].shape[0]
        return self


def layers_to_device(policy_spec, device="cuda") -> List[dict]:
    """PolicySpec (workloads.py) -> list of layer dicts holding cuda tensors."""
    out = []
    for l in policy_spec.layers:
        d = {"weight": torch.from_numpy(l.weight).to(device).contiguous()}
        if l.bias is not None:
            d["bias"] = torch.from_numpy(l.bias).to(device).contiguous()
        if l.kind == "conv":
            d["stride"], d["in_hw"] = l.stride, l.in_hw
        if getattr(l, "per_channel", False):
            d["per_channel"] = True
        out.append(d)
    return out
