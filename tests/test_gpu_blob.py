"""Packed policy blob (the paper's quantized communication): export from one policy, import into
another of the same architecture, identical results; the blob is about a quarter of the fp32 weights."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import oracle as O                      # noqa: E402
from paper_1910_01055_b200 import binding as B      # noqa: E402
from paper_1910_01055_b200 import workloads as W    # noqa: E402


def _matches_checker(spec, obs_np, out, actions):
    """the importing policy against the CPU checker run on the SENDER's fp32 weights"""
    qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
    y_ref, act_ref, _ = O.forward(qp, obs_np)
    y = out.cpu().numpy()
    assert np.all(np.abs(y - y_ref) <= 1e-5 * np.abs(y_ref) + 1e-30), float(np.abs(y - y_ref).max())
    if spec.head != "tanh":
        assert np.array_equal(y, y_ref)
    if act_ref is not None:
        assert np.array_equal(actions.cpu().numpy(), act_ref)


def _policy(spec):
    return B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(B.layers_to_device(spec), spec.input_ranges)


def _specs(kind, seed):
    if kind == "mlp":
        return W.calibrate(W.mlp_policy("m", [67, 256, 256, 256, 21], seed=seed, nonzero_bias=True), 128, seed=seed)
    if kind == "wide":
        return W.calibrate(W.mlp_policy("w", [128, 1024, 1024, 32], seed=seed), 128, seed=seed)
    if kind == "conv":      # tensor-core conv path
        return W.calibrate(W.dqn_policy("c", seed=seed, in_hw=(44, 52), channels=(4, 32, 64, 64), fc_hidden=64, n_actions=18, nonzero_bias=True), 32, seed=seed)
    return W.calibrate(W.dqn_policy("g", seed=seed, in_hw=(36, 36), channels=(2, 8, 16, 16), fc_hidden=32, n_actions=5), 32, seed=seed)   # generic path


@pytest.mark.parametrize("kind", ["mlp", "wide", "conv", "generic"])
def test_blob_round_trip(kind):
    from paper_1910_01055_b200 import build
    build.build()
    src_spec, dst_spec = _specs(kind, 3), _specs(kind, 4)
    dst_spec.input_ranges = src_spec.input_ranges            # activation ranges are part of the architecture's calibration
    src, dst = _policy(src_spec), _policy(dst_spec)
    obs_np = W.make_obs(src_spec, 300, seed=5)
    obs = torch.from_numpy(obs_np).cuda()
    want, want_act = src.forward(obs)
    other, _ = dst.forward(obs)
    assert not torch.equal(want, other)                      # different weights before the import
    n = B.actorq_policy_blob_bytes(src.handle)
    fp32_bytes = sum(l.weight.nbytes for l in src_spec.layers)
    codes = sum(l.weight.size for l in src_spec.layers)
    assert n == B.actorq_policy_blob_bytes(dst.handle)
    assert codes <= n <= codes + 64 + 48 * len(src_spec.layers) + sum(16 + 12 * ((l.weight.shape[0] + 127) // 128 * 128) for l in src_spec.layers) + 16 * len(src_spec.layers)
    if kind == "wide":
        assert n < 0.26 * fp32_bytes                         # "4x smaller" plus a little metadata
    blob = torch.empty(n, dtype=torch.uint8, device="cuda")
    B.actorq_policy_export_blob(src.handle, blob)
    wire = blob.clone()                                      # the broadcast: one device buffer
    B.actorq_policy_import_blob(dst.handle, wire)
    got, got_act = dst.forward(obs)
    torch.cuda.synchronize()
    assert dst.status() == B.OK and src.status() == B.OK
    assert torch.equal(got, want)
    if want_act is not None:
        assert torch.equal(got_act, want_act)
    _matches_checker(src_spec, obs_np, got, got_act)
    for i, l in enumerate(src_spec.layers):                   # codes, delta and zero-point arrived too
        a = torch.empty(l.weight.shape, dtype=torch.int8, device="cuda")
        b = torch.empty_like(a)
        sa = B.actorq_policy_export_layer(src.handle, i, a)
        sb = B.actorq_policy_export_layer(dst.handle, i, b)
        assert sa == sb and torch.equal(a, b)
    src.close()
    dst.close()


def test_blob_rejects_wrong_size_and_foreign_architecture():
    a, b = _policy(_specs("mlp", 3)), _policy(_specs("wide", 3))
    na, nb = B.actorq_policy_blob_bytes(a.handle), B.actorq_policy_blob_bytes(b.handle)
    blob = torch.zeros(max(na, nb), dtype=torch.uint8, device="cuda")
    B.actorq_policy_export_blob(a.handle, blob)
    with pytest.raises(B.ActorQError) as e:
        B.actorq_policy_import_blob(b.handle, blob[:na])                  # size of another architecture
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.ActorQError):
        B.actorq_policy_export_blob(a.handle, blob[:na - 16])             # too small a buffer
    damaged = blob[:na].clone()
    damaged[0] ^= 0xFF                                                    # break the magic
    B.actorq_policy_import_blob(a.handle, damaged)
    torch.cuda.synchronize()
    assert a.status() == B.ERR_INVALID_ARG
    B.actorq_policy_import_blob(a.handle, blob[:na].clone())              # a good blob restores it
    torch.cuda.synchronize()
    assert a.status() == B.OK
    a.close()
    b.close()


def test_blob_round_trip_per_channel_policy():
    """A policy quantized per output channel travels with its per-channel deltas, zero-points and
    multipliers: after the import the receiving policy computes what the sender computes."""
    def spec(seed):
        s = W.dqn_policy("p", seed=seed, in_hw=(36, 36), channels=(2, 8, 16, 16), fc_hidden=32, n_actions=5, nonzero_bias=True)
        for l in s.layers:
            l.per_channel = True
        return W.calibrate(s, 32, seed=seed)
    src_spec, dst_spec = spec(3), spec(4)
    dst_spec.input_ranges = src_spec.input_ranges
    src, dst = _policy(src_spec), _policy(dst_spec)
    obs_np = W.make_obs(src_spec, 100, seed=5)
    obs = torch.from_numpy(obs_np).cuda()
    want, want_act = src.forward(obs)
    n = B.actorq_policy_blob_bytes(src.handle)
    blob = torch.empty(n, dtype=torch.uint8, device="cuda")
    B.actorq_policy_export_blob(src.handle, blob)
    B.actorq_policy_import_blob(dst.handle, blob.clone())
    got, got_act = dst.forward(obs)
    torch.cuda.synchronize()
    assert dst.status() == B.OK and torch.equal(got, want) and torch.equal(got_act, want_act)
    _matches_checker(src_spec, obs_np, got, got_act)
    for i, l in enumerate(src_spec.layers):
        a = torch.empty(l.weight.shape, dtype=torch.int8, device="cuda")
        b = torch.empty_like(a)
        sa, za = B.actorq_policy_export_layer_channels(src.handle, i, a)
        sb, zb = B.actorq_policy_export_layer_channels(dst.handle, i, b)
        assert torch.equal(a, b) and (sa == sb).all() and (za == zb).all()
    src.close(); dst.close()
