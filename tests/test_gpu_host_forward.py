"""actorq_policy_forward_host: chunked, pipelined forward on host buffers, held bit for bit against
actorq_policy_forward on device buffers and, on sampled rows, against the CPU checker."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_1910_01055_b200 import binding as B
from paper_1910_01055_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_1910_01055_b200 import build
    build.build()
    B.load()


def _policy(spec):
    return B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(B.layers_to_device(spec), spec.input_ranges)


def _matches_checker(spec, obs_np, out_host, actions_host=None, max_rows=400):
    """rows spread over every chunk of the call (first, last, and evenly spaced) against the checker"""
    n = obs_np.shape[0]
    idx = np.unique(np.concatenate([np.arange(min(n, 3)), np.arange(max(0, n - 3), n),
                                    np.linspace(0, n - 1, min(n, max_rows)).astype(np.int64)]))
    qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
    y_ref, act_ref, _ = O.forward(qp, obs_np[idx])
    y = out_host.numpy()[idx]
    assert np.all(np.abs(y - y_ref) <= 1e-5 * np.abs(y_ref) + 1e-30), float(np.abs(y - y_ref).max())
    if act_ref is not None:
        assert np.array_equal(y, y_ref) and np.array_equal(actions_host.numpy()[idx], act_ref)


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("Bsz", [1, 300, 31232, 70000])       # one chunk is 31232 rows of 67 floats
def test_host_forward_matches_device_forward_mlp(Bsz, pinned):
    spec = W.build_config("d4pg_humanoid")
    pol = _policy(spec)
    obs = torch.from_numpy(W.make_obs(spec, Bsz, seed=5))
    ref, _ = pol.forward(obs.cuda())
    torch.cuda.synchronize()
    out = torch.empty((Bsz, spec.out_dim), dtype=torch.float32)
    if pinned:
        obs, out = obs.pin_memory(), out.pin_memory()
    for _ in range(2):                                          # the second call reuses the staging slots
        out.zero_()
        B.actorq_policy_forward_host(pol.handle, obs, out)
        torch.cuda.synchronize()
        assert pol.status() == B.OK
        assert torch.equal(out, ref.cpu())
    _matches_checker(spec, obs.numpy(), out)
    pol.close()


def test_host_forward_conv_policy_with_actions_and_requantize_between():
    spec = W.calibrate(W.dqn_policy("c", in_hw=(84, 84)), 16)
    layers_dev = B.layers_to_device(spec)
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(layers_dev, spec.input_ranges)
    Bsz = 600                                                   # 256-row chunks: two full, one ragged
    obs = torch.from_numpy(W.make_obs(spec, Bsz, seed=6)).pin_memory()
    out = torch.empty((Bsz, spec.out_dim), dtype=torch.float32).pin_memory()
    act = torch.empty((Bsz,), dtype=torch.int32).pin_memory()
    for _ in range(2):
        pol.quantize(layers_dev, spec.input_ranges)             # enqueued before the call: must run first
        B.actorq_policy_forward_host(pol.handle, obs, out, act)
        torch.cuda.synchronize()
        ref, ref_act = pol.forward(obs.cuda())
        torch.cuda.synchronize()
        assert pol.status() == B.OK
        assert torch.equal(out, ref.cpu()) and torch.equal(act, ref_act.cpu())
    _matches_checker(spec, obs.numpy(), out, act, max_rows=12)
    pol.close()


def test_host_forward_argument_checks():
    spec = W.build_config("d4pg_tiny")
    pol = _policy(spec)
    lib = B.load()
    assert lib.actorq_policy_forward_host(pol.handle, None, 4, None, None, None) == B.ERR_INVALID_ARG
    assert lib.actorq_policy_forward_host(pol.handle, None, 0, None, None, None) == B.OK
    assert lib.actorq_policy_forward_host(None, None, 0, None, None, None) == B.ERR_INVALID_ARG
    pol.close()
