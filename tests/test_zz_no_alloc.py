"""The allocation-free forward against the ordinary one (and the CPU checker), through the C ABI.

Some deployments cannot let the library allocate once the actor loop is live: the learner's
framework already owns the device's memory pool, and a raw cudaMalloc both risks failing and stalls
every stream on the device while it runs.  actorq_policy_forward_noalloc serves them from a fixed
scratch array inside the library.  Here it must reproduce actorq_policy_forward on two calls in a
row (the second one re-uses whatever the first left in the shared array), for a fully connected
and for a convolutional policy, and must refuse a batch that does not fit.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import oracle as O                      # noqa: E402
from paper_1910_01055_b200 import binding as B      # noqa: E402
from paper_1910_01055_b200 import workloads as W    # noqa: E402

REL_TOL = 1e-5    # the tolerance of the other GPU parity tests (only the tanh head can differ at all)


def _both(pol, spec, obs_np):
    obs = torch.from_numpy(obs_np).cuda()
    ref, ref_act = pol.forward(obs)
    out = torch.full_like(ref, float("nan"))
    act = torch.full_like(ref_act, -1) if ref_act is not None else None
    B.actorq_policy_forward_noalloc(pol.handle, obs, out, act)
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    r, o = ref.cpu().numpy(), out.cpu().numpy()
    assert np.all(np.abs(o - r) <= REL_TOL * np.abs(r) + 1e-30), float(np.abs(o - r).max())
    if ref_act is not None:
        assert torch.equal(act, ref_act)
    # and against the CPU checker directly, so that this entry point does not lean on the other one
    qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
    y_ref, act_ref, _ = O.forward(qp, obs_np)
    assert np.all(np.abs(o - y_ref) <= REL_TOL * np.abs(y_ref) + 1e-30), float(np.abs(o - y_ref).max())
    if act_ref is not None:
        assert np.array_equal(o, y_ref) and np.array_equal(act.cpu().numpy(), act_ref)


@pytest.mark.parametrize("kind", ["mlp", "conv"])
def test_noalloc_matches_forward_twice_in_a_row(kind):
    from paper_1910_01055_b200 import build
    build.build()
    if kind == "mlp":
        spec = W.build_config("d4pg_humanoid")
        batches = [777, 130]
    else:
        spec = W.calibrate(W.dqn_policy("c", seed=9, in_hw=(44, 44), channels=(4, 16, 32, 32), fc_hidden=64, n_actions=6), 32, seed=9)
        batches = [65, 200]
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(B.layers_to_device(spec), spec.input_ranges)
    for i, bsz in enumerate(batches):                      # two calls in a row on the shared scratch
        _both(pol, spec, W.make_obs(spec, bsz, seed=9, index=i))
    pol.close()


def test_noalloc_rejects_a_batch_beyond_the_fixed_scratch():
    spec = W.calibrate(W.mlp_policy("t", [8, 32, 4], seed=2), 64, seed=2)
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(B.layers_to_device(spec), spec.input_ranges)
    limit = (B.NOALLOC_SCRATCH_BYTES // 2) // 32           # widest layer has 32 elements per row
    obs = torch.zeros((limit + 1, 8), dtype=torch.float32, device="cuda")
    out = torch.empty((limit + 1, 4), dtype=torch.float32, device="cuda")
    with pytest.raises(B.ActorQError) as e:
        B.actorq_policy_forward_noalloc(pol.handle, obs, out)
    assert e.value.code == B.ERR_SCRATCH_LIMIT
    B.actorq_policy_forward_noalloc(pol.handle, obs[:limit], out[:limit])     # exactly at the limit is fine
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    ref, _ = pol.forward(obs[:limit])
    assert torch.equal(ref, out[:limit])
    pol.close()
