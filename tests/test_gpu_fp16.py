"""The fp16 actor (the paper's q = 16 policies) through the C ABI against the CPU checker.

Tolerance (there is no bit-exact contract: the tensor core sums binary32 partial products in an order of its
own).  The checker sums in double and rounds once.  Per layer the GPU's accumulation differs from the exact sum
by at most ~K * 2^-24 of the sum of magnitudes; where that moves a hidden activation across a rounding boundary
the binary16 value differs by one step, 2^-10 relative.  Propagating "every activation off by one step" through
the layers bounds the difference of an output by  sum_l 2^-10 * (|W_L| ... |W_{l+1}| |a_l|)  -- computed below
from the checker's own activations -- plus the binary32 accumulation terms; the observed differences are a few
1e-5, far inside."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import oracle as O                                    # noqa: E402
from paper_1910_01055_b200 import binding as B                    # noqa: E402
from paper_1910_01055_b200 import workloads as W                  # noqa: E402


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_1910_01055_b200 import build
    build.build()
    B.load()


def _bound(spec, obs_rows, trace_rows):
    """per output: sum over layers of one binary16 step of that layer's input, pushed through |W| of the rest,
    plus K * 2^-22 of the magnitudes for the binary32 accumulations"""
    n = len(spec.layers)
    w16 = [np.abs(O.cast_fp16(l.weight).astype(np.float64)) for l in spec.layers]
    acts = [np.abs(O.cast_fp16(obs_rows).astype(np.float64))] + [np.abs(t.astype(np.float64)) for t in trace_rows[:-1]]
    total = np.zeros((obs_rows.shape[0], spec.layers[-1].weight.shape[0]))
    for l in range(n):
        e = acts[l] * (2.0 ** -10 if l > 0 else 0.0)               # the observations are rounded identically on both sides
        for m in range(l, n):
            e = e @ w16[m].T + (acts[m] @ w16[m].T) * (spec.layers[m].weight.shape[1] * 2.0 ** -22 if m == l else 0.0)
        total += e
    return total + 1e-6


@pytest.mark.parametrize("dims,head,Bsz", [([67, 256, 256, 256, 21], "tanh", 4097), ([128, 1024, 1024, 32], "tanh", 700),
                                           ([24, 96, 200, 6], "argmax", 300), ([10, 2048, 2048, 4], "linear", 257),
                                           ([3, 16, 2], "tanh", 1), ([70, 5], "linear", 130)])
def test_fp16_actor_matches_checker(dims, head, Bsz):
    spec = W.mlp_policy("h", dims, seed=77, head=head, nonzero_bias=True)
    layers_dev = B.layers_to_device(spec)
    handle = B.actorq_cast_params_fp16(layers_dev, head, "f32")
    obs = W.make_obs(spec, Bsz, seed=77)
    obs_d = torch.from_numpy(obs).cuda()
    out = torch.empty((Bsz, dims[-1]), dtype=torch.float32, device="cuda")
    act = torch.empty((Bsz,), dtype=torch.int32, device="cuda") if head == "argmax" else None
    B.actorq_policy_forward(handle, obs_d, out, act)
    torch.cuda.synchronize()
    assert B.actorq_policy_last_device_status(handle) == B.OK
    y_ref, act_ref, trace = O.forward_fp16(spec.layers, obs, head)
    got = out.cpu().numpy()
    diff = np.abs(got.astype(np.float64) - y_ref.astype(np.float64))
    assert np.all(diff <= _bound(spec, obs, trace)), float(diff.max())
    assert diff.max() < 2e-3 * max(1.0, float(np.abs(y_ref).max()))
    if act_ref is not None:          # greedy actions agree wherever the two best Q-values are further apart than the outputs differ
        srt = np.sort(y_ref, axis=1)
        clear = (srt[:, -1] - srt[:, -2]) > 2 * diff.max(axis=1) + 1e-7
        assert clear.mean() > 0.9 and np.array_equal(act.cpu().numpy()[clear], act_ref[clear])
    # re-cast in place after a weight update (a broadcast): same handle, new results match the checker again
    spec.layers[0].weight += np.float32(0.01)
    layers_dev[0]["weight"].copy_(torch.from_numpy(spec.layers[0].weight))
    before = handle.value
    handle = B.actorq_cast_params_fp16(layers_dev, head, "f32", handle)
    assert handle.value == before
    B.actorq_policy_forward(handle, obs_d, out, act)
    torch.cuda.synchronize()
    y2, _, trace2 = O.forward_fp16(spec.layers, obs, head)
    diff2 = np.abs(out.cpu().numpy().astype(np.float64) - y2.astype(np.float64))
    assert np.all(diff2 <= _bound(spec, obs, trace2)) and np.abs(y2 - y_ref).max() > 0
    # a row's result does not depend on the batch
    one = torch.empty((1, dims[-1]), dtype=torch.float32, device="cuda")
    B.actorq_policy_forward(handle, obs_d[Bsz // 2: Bsz // 2 + 1].clone(), one, act[:1].clone() if act is not None else None)
    torch.cuda.synchronize()
    assert torch.equal(one[0], out[Bsz // 2])
    B.actorq_free(handle)


def test_fp16_policy_rejects_int8_only_calls_and_conv_policies():
    spec = W.mlp_policy("h", [8, 32, 4], seed=2, head="tanh")
    layers_dev = B.layers_to_device(spec)
    handle = B.actorq_cast_params_fp16(layers_dev, "tanh", "f32")
    with pytest.raises(B.ActorQError) as e:
        B.actorq_policy_set_fused_variant(handle, 2)
    assert e.value.code == B.ERR_UNSUPPORTED
    w_q = torch.empty((32, 8), dtype=torch.int8, device="cuda")
    with pytest.raises(B.ActorQError):
        B.actorq_policy_export_layer(handle, 0, w_q)
    with pytest.raises(B.ActorQError) as e:
        B.actorq_quantize_params(layers_dev, [(-1.0, 1.0), (0.0, 1.0)], "tanh", "f32", handle)
    assert e.value.code == B.ERR_INVALID_ARG
    # exploration noise works on an fp16 policy too (drawn by the kernel behind the forward)
    obs = torch.from_numpy(W.make_obs(spec, 40, seed=2)).cuda()
    plain = torch.empty((40, 4), device="cuda")
    noisy = torch.empty((40, 4), device="cuda")
    B.actorq_policy_forward(handle, obs, plain)
    sigma = torch.full((40,), 0.1, device="cuda")
    B.actorq_policy_forward_explore_seeded(handle, obs, sigma, 5, noisy)
    torch.cuda.synchronize()
    z = O.exploration_normals(5, 0, 40, 4).astype(np.float32)
    want = O.explore(plain.cpu().numpy(), sigma.cpu().numpy(), z)
    assert np.abs(noisy.cpu().numpy() - want).max() <= 2e-6
    B.actorq_free(handle)
