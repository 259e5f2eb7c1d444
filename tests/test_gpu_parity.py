"""GPU-vs-checker parity through the C ABI (run with -m gpu on a B200).

Bars: int8 weight codes, zero-points, int32 accumulators and int8 hidden activations are
compared bit for bit; deltas must be equal as binary32 numbers; final fp32 outputs within 1e-5
relative (only tanh differs between the two sides: the checker rounds a double tanh, the GPU
uses single-precision tanhf; linear / Q-value outputs are bit-exact); argmax actions identical.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from oracle import oracle as O                                    # noqa: E402
from paper_1910_01055_b200 import binding as B                    # noqa: E402
from paper_1910_01055_b200 import workloads as W                  # noqa: E402

REL_TOL = 1e-5


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_1910_01055_b200 import build
    build.build()
    B.load()
    O.lib()


def _quantize_both(spec):
    layers_dev = B.layers_to_device(spec)
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(layers_dev, spec.input_ranges)
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
    return pol, qp, layers_dev


def _check_weights(pol, qp, spec):
    for i, (l, ql) in enumerate(zip(spec.layers, qp.layers)):
        w_q = torch.empty(l.weight.shape, dtype=torch.int8, device="cuda")
        if ql.per_channel:
            s, z = B.actorq_policy_export_layer_channels(pol.handle, i, w_q)
            assert np.array_equal(s, ql.s_w) and np.array_equal(z, ql.z_w), i
            assert np.array_equal(w_q.cpu().numpy(), ql.w_q), i
            continue
        s, z = B.actorq_policy_export_layer(pol.handle, i, w_q)
        assert np.float32(s) == ql.s_w, (i, s, ql.s_w)
        assert z == ql.z_w, (i, z, ql.z_w)
        got = w_q.cpu().numpy()
        assert np.array_equal(got, ql.w_q), (i, int((got != ql.w_q).sum()))


def _check_forward(pol, qp, spec, obs, sample=None, check_layers=True):
    """GPU on the full batch; checker on `sample` rows (all rows if None)."""
    obs_dev = torch.from_numpy(obs).cuda()
    out, actions = pol.forward(obs_dev)
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    idx = np.arange(obs.shape[0]) if sample is None else np.asarray(sample)
    y_ref, act_ref, trace = O.forward(qp, obs[idx])
    n = len(spec.layers)
    if check_layers:
        for i in range(n):
            acc = torch.empty((obs.shape[0], spec.layers[i].out_features), dtype=torch.int32, device="cuda")
            act = torch.empty((obs.shape[0], spec.layers[i].out_features), dtype=torch.int8, device="cuda") if i + 1 < n else None
            out_d = torch.empty_like(out)
            actions_d = torch.empty_like(actions) if actions is not None else None
            B.actorq_policy_forward_debug(pol.handle, obs_dev, out_d, actions_d, i, acc, act)
            torch.cuda.synchronize()
            assert pol.status() == B.OK
            acc_g = acc.cpu().numpy()[idx]
            ref_acc = trace[i][0].reshape(len(idx), -1)
            assert np.array_equal(acc_g, ref_acc), (i, "acc", int((acc_g != ref_acc).sum()), acc_g.ravel()[:8], ref_acc.ravel()[:8])
            if act is not None:
                act_g = act.cpu().numpy()[idx]
                ref_act = trace[i][1].reshape(len(idx), -1)
                assert np.array_equal(act_g, ref_act), (i, "act", int((act_g != ref_act).sum()))
            assert torch.equal(out_d, out)          # the debug call runs the same kernels
    y = out.cpu().numpy()[idx]
    if spec.head == "tanh":
        assert np.all(np.abs(y - y_ref) <= REL_TOL * np.abs(y_ref) + 1e-30), np.abs(y - y_ref).max()
    else:
        assert np.array_equal(y, y_ref)
    if spec.head == "argmax":
        assert np.array_equal(actions.cpu().numpy()[idx], act_ref)
    return out, actions


# ---- the five configurations -------------------------------------------------------------

def test_config1_d4pg_tiny():
    spec = W.build_config("d4pg_tiny")
    pol, qp, _ = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    _check_forward(pol, qp, spec, W.make_obs(spec, 64))
    pol.close()


def test_config2_d4pg_humanoid():
    spec = W.build_config("d4pg_humanoid")
    pol, qp, _ = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    _check_forward(pol, qp, spec, W.make_obs(spec, 4096))
    pol.close()


def test_config3_mlp_wide_full_batch_sampled():
    spec = W.build_config("mlp_wide")
    pol, qp, _ = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    Bsz = 65536
    obs = W.make_obs(spec, Bsz)
    rng = np.random.default_rng(0)
    sample = np.unique(np.concatenate([np.arange(0, 130), np.arange(Bsz - 130, Bsz), rng.integers(0, Bsz, 256)]))
    _check_forward(pol, qp, spec, obs, sample)
    pol.close()


def test_config4_dqn_conv_sampled():
    spec = W.build_config("dqn_conv")
    pol, qp, _ = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    Bsz = 1024
    obs = W.make_obs(spec, Bsz)
    sample = np.unique(np.concatenate([np.arange(0, 4), np.arange(Bsz - 4, Bsz), np.random.default_rng(1).integers(0, Bsz, 16)]))
    _check_forward(pol, qp, spec, obs, sample)
    pol.close()


def test_config5_actor_sweep_with_requantization():
    """config-2 network, batch sweep, weights perturbed and re-quantized in place between rounds"""
    spec = W.build_config("actor_sweep")
    pol, qp, layers_dev = _quantize_both(spec)
    for rnd, Bsz in enumerate([1, 16, 256, 4096, 65536, 262144]):
        if rnd:
            W.perturb_weights(spec, rnd)
            for d, l in zip(layers_dev, spec.layers):
                d["weight"].copy_(torch.from_numpy(l.weight))
            handle_before = pol.handle.value
            pol.quantize(layers_dev, spec.input_ranges)          # in place: same handle
            assert pol.handle.value == handle_before
            qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
            _check_weights(pol, qp, spec)
        obs = W.make_obs(spec, Bsz, index=rnd)
        sample = None
        if Bsz > 4096:
            sample = np.unique(np.concatenate([np.arange(0, 130), np.arange(Bsz - 130, Bsz),
                                               np.random.default_rng(rnd).integers(0, Bsz, 1024)]))
        _check_forward(pol, qp, spec, obs, sample, check_layers=(Bsz <= 65536))
    pol.close()


# ---- structure and edge cases ----------------------------------------------------------------

@pytest.mark.parametrize("dims,head", [([24, 256, 256, 256, 6], "tanh"), ([67, 256, 256, 256, 21], "tanh"),
                                       ([5, 48, 7], "linear"), ([33, 100, 130, 9], "argmax"),
                                       ([128, 1024, 1024, 32], "tanh"), ([3, 4], "linear")])
@pytest.mark.parametrize("Bsz", [1, 2, 127, 128, 129, 4097])
def test_ragged_batches_and_row_independence(dims, head, Bsz):
    spec = W.calibrate(W.mlp_policy("t", dims, seed=3, head=head, nonzero_bias=True), 256, seed=3)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, Bsz, seed=3)
    out, _ = _check_forward(pol, qp, spec, obs, check_layers=(Bsz in (1, 129)))
    # a row's result does not depend on the batch it travels in
    sub = torch.from_numpy(obs[Bsz // 2: Bsz // 2 + 1]).cuda()
    out1, _ = pol.forward(sub)
    torch.cuda.synchronize()
    assert torch.equal(out1[0], out[Bsz // 2])
    pol.close()


def test_small_conv_nets():
    for (hw, ch, fc, nact, Bsz) in [((36, 36), (2, 8, 16, 16), 32, 5, 3), ((44, 52), (4, 32, 64, 64), 64, 18, 130)]:
        spec = W.calibrate(W.dqn_policy("c", seed=5, n_actions=nact, in_hw=hw, channels=ch, fc_hidden=fc,
                                        nonzero_bias=True), 32, seed=5)
        pol, qp, _ = _quantize_both(spec)
        _check_weights(pol, qp, spec)
        _check_forward(pol, qp, spec, W.make_obs(spec, Bsz, seed=5))
        pol.close()


def test_quantizer_edge_tensors():
    """all-zero tensor, all-positive, all-negative, odd sizes, unaligned row length"""
    rng = np.random.default_rng(8)
    ws = [np.zeros((4, 7), np.float32), np.abs(rng.standard_normal((9, 13))).astype(np.float32) + 0.1,
          -np.abs(rng.standard_normal((6, 5))).astype(np.float32), rng.standard_normal((1, 1)).astype(np.float32),
          (rng.standard_normal((300, 67)) * 1e-12).astype(np.float32), (rng.standard_normal((17, 4100)) * 1e6).astype(np.float32)]
    for w in ws:
        spec = W.PolicySpec("e", [W.LayerSpec("fc", w, None)], "linear", "f32", [(-1.0, 1.0)])
        pol, qp, _ = _quantize_both(spec)
        _check_weights(pol, qp, spec)
        pol.close()


def test_large_tensor_streaming_quantizer():
    w = np.random.default_rng(4).standard_normal((4096, 8192)).astype(np.float32)
    spec = W.PolicySpec("big", [W.LayerSpec("fc", w, None)], "linear", "f32", [(-1.0, 1.0)])
    pol, qp, _ = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    pol.close()


def test_saturating_and_nan_observations():
    spec = W.calibrate(W.mlp_policy("t", [24, 256, 256, 6], seed=2), 256, seed=2)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, 130, seed=2) * 50.0                  # far outside the calibrated range
    obs[0, :] = np.nan
    obs[1, 0], obs[1, 1] = np.inf, -np.inf
    obs[2, :] = 1e38
    _check_forward(pol, qp, spec, obs)
    pol.close()


def test_nonfinite_weight_is_reported_not_trapped():
    spec = W.calibrate(W.mlp_policy("t", [8, 32, 4], seed=2), 64, seed=2)
    layers_dev = B.layers_to_device(spec)
    layers_dev[1]["weight"][3, 5] = float("nan")
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(layers_dev, spec.input_ranges)
    torch.cuda.synchronize()
    assert pol.status() == B.ERR_NONFINITE
    assert pol.status() == B.OK                                   # cleared by the read
    layers_dev[1]["weight"][3, 5] = 0.25
    pol.quantize(layers_dev, spec.input_ranges)                   # the context is still usable
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    spec.layers[1].weight[3, 5] = 0.25
    qp = O.quantize_policy(spec.layers, spec.input_ranges, spec.head, spec.obs_dtype)
    _check_weights(pol, qp, spec)
    pol.close()


def test_requantize_checks_architecture_and_empty_batch():
    spec = W.calibrate(W.mlp_policy("t", [8, 32, 4], seed=2), 64, seed=2)
    pol, qp, layers_dev = _quantize_both(spec)
    other = W.calibrate(W.mlp_policy("t", [8, 48, 4], seed=2), 64, seed=2)
    with pytest.raises(B.ActorQError) as e:
        B.actorq_quantize_params(B.layers_to_device(other), other.input_ranges, "tanh", "f32", pol.handle)
    assert e.value.code == B.ERR_INVALID_ARG
    empty = torch.empty((0, 8), dtype=torch.float32, device="cuda")
    out = torch.empty((0, 4), dtype=torch.float32, device="cuda")
    B.actorq_policy_forward(pol.handle, empty, out)
    # re-quantizing in place gives the same result as a fresh handle
    obs = torch.from_numpy(W.make_obs(spec, 77)).cuda()
    y1, _ = pol.forward(obs)
    pol.quantize(layers_dev, spec.input_ranges)
    y2, _ = pol.forward(obs)
    fresh, _, _ = _quantize_both(spec)
    y3, _ = fresh.forward(obs)
    torch.cuda.synchronize()
    assert torch.equal(y1, y2) and torch.equal(y1, y3)
    pol.close()
    fresh.close()


def test_requantize_conversion_paths():
    """The fused epilogue converts int32 -> float with a bit trick that is exact up to 2^22 and only
    enabled when larger accumulators are sure to clamp; exercise (a) accumulators far above 2^22 in
    both directions, (b) a multiplier too small for the trick, (c) biases too large for it."""
    rng = np.random.default_rng(21)
    # (a) all-positive / all-negative wide layers driven by saturated inputs
    for sign in (1.0, -1.0):
        spec = W.mlp_policy("big", [128, 1024, 1024, 8], seed=4, head="linear")
        spec.layers[0].weight = np.abs(spec.layers[0].weight)
        spec.layers[1].weight = (sign * np.abs(spec.layers[1].weight)).astype(np.float32)
        W.calibrate(spec, 128, seed=4)
        pol, qp, _ = _quantize_both(spec)
        obs = np.abs(W.make_obs(spec, 200, seed=4)) * 100.0
        _, _, trace = O.forward(qp, obs)
        assert np.abs(trace[1][0]).max() > 2 ** 23
        _check_forward(pol, qp, spec, obs)
        pol.close()
    # (b) a hidden range so wide that M < 2^-13
    spec = W.calibrate(W.mlp_policy("tinyM", [64, 256, 256, 5], seed=6, head="linear"), 128, seed=6)
    spec.input_ranges[1] = (0.0, 3.0e4)
    pol, qp, _ = _quantize_both(spec)
    assert float(qp.layers[0].M) < 2.0 ** -13
    _check_forward(pol, qp, spec, W.make_obs(spec, 300, seed=6) * 200.0)
    pol.close()
    # (c) biases whose integer image exceeds 2^29
    spec = W.mlp_policy("bigbias", [64, 256, 256, 5], seed=7, head="linear")
    spec.layers[0].bias = (rng.standard_normal(256) * 3.0e4).astype(np.float32)
    W.calibrate(spec, 128, seed=7)
    spec.input_ranges[1] = (0.0, 4.0)
    pol, qp, _ = _quantize_both(spec)
    assert np.abs(qp.layers[0].bias_q).max() > 2 ** 29
    _check_forward(pol, qp, spec, W.make_obs(spec, 300, seed=7))
    pol.close()


def test_requantize_clamp_modes():
    """Hidden layers whose next zero-point is not -128, or whose multiplier is large, take the
    float-clamp path instead of the saturating pack; heavy saturation exercises both clamps."""
    for rng_hidden in [(-1.0, 4.0), (0.0, 0.02), (0.0, 3.0)]:
        spec = W.calibrate(W.mlp_policy("m", [40, 256, 192, 7], seed=11, head="linear", nonzero_bias=True), 128, seed=11)
        spec.input_ranges[1] = rng_hidden
        pol, qp, _ = _quantize_both(spec)
        obs = W.make_obs(spec, 300, seed=11) * 3.0
        _check_forward(pol, qp, spec, obs)
        pol.close()


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("dims,head,Bsz", [([24, 256, 256, 256, 6], "tanh", 200),
                                           ([67, 256, 256, 256, 21], "tanh", 1500),
                                           ([50, 416, 300, 160, 9], "linear", 700),      # chunk halves that straddle weight tiles
                                           ([33, 96, 520, 1000, 40, 3], "tanh", 385),    # narrow, ragged and 5 layers
                                           ([128, 1024, 1024, 12], "linear", 513)])
def test_both_fused_kernels_match_checker(variant, dims, head, Bsz):
    """The single-CTA fused kernel (variant 1) and the CTA-pair kernel (variant 2, signed first layer,
    unsigned hidden codes) are each held against the checker: accumulators and codes of every layer,
    outputs, and the two kernels' outputs against each other bit for bit."""
    spec = W.calibrate(W.mlp_policy("v", dims, seed=31, head=head, nonzero_bias=(len(dims) % 2 == 0)), 128, seed=31)
    pol, qp, _ = _quantize_both(spec)
    B.actorq_policy_set_fused_variant(pol.handle, variant)
    obs = W.make_obs(spec, Bsz, seed=31)
    out, _ = _check_forward(pol, qp, spec, obs)
    B.actorq_policy_set_fused_variant(pol.handle, 3 - variant)
    other, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    assert torch.equal(out, other)
    pol.close()


def test_fused_variant_switch_rejects_bad_arguments():
    spec = W.build_config("d4pg_tiny")
    pol, _, _ = _quantize_both(spec)
    with pytest.raises(B.ActorQError):
        B.actorq_policy_set_fused_variant(pol.handle, 7)
    B.actorq_policy_set_fused_variant(pol.handle, 0)
    pol.close()
    conv = W.calibrate(W.dqn_policy("c", in_hw=(44, 44), channels=(4, 16, 32, 32), fc_hidden=64, n_actions=6), 16)
    polc, _, _ = _quantize_both(conv)
    with pytest.raises(B.ActorQError):
        B.actorq_policy_set_fused_variant(polc.handle, 2)
    polc.close()


@pytest.mark.parametrize("which", ["conv_layers", "all_layers", "mlp", "mlp_mixed"])
def test_per_channel_quantization_matches_checker(which):
    """Per-output-channel weight quantization (the paper's scheme for convolutional layers): codes,
    per-channel deltas and zero-points, every layer's accumulators and codes, outputs and actions."""
    if which == "mlp":
        spec = W.mlp_policy("pc", [40, 96, 130, 7], seed=51, head="tanh", nonzero_bias=True)
        for l in spec.layers:
            l.weight *= np.linspace(0.05, 3.0, l.weight.shape[0], dtype=np.float32).reshape(-1, 1)   # rows of very different size
            l.per_channel = True
        W.calibrate(spec, 128, seed=51)
        obs = W.make_obs(spec, 300, seed=51)
    elif which == "mlp_mixed":       # wider than the fused kernels, per-channel and per-tensor layers alternating
        spec = W.mlp_policy("pcm", [30, 1100, 200, 9], seed=53, head="linear", nonzero_bias=True)
        for i, l in enumerate(spec.layers):
            if i != 1:
                l.weight *= np.linspace(0.1, 2.0, l.weight.shape[0], dtype=np.float32).reshape(-1, 1)
                l.per_channel = True
        W.calibrate(spec, 128, seed=53)
        obs = W.make_obs(spec, 515, seed=53)
    else:
        spec = W.dqn_policy("pc", in_hw=(44, 44), channels=(4, 16, 32, 32), fc_hidden=64, n_actions=6, nonzero_bias=True)
        for l in spec.layers:
            if l.kind == "conv" or which == "all_layers":
                l.per_channel = True
        W.calibrate(spec, 16)
        obs = W.make_obs(spec, 37, seed=52)
    pol, qp, layers_dev = _quantize_both(spec)
    _check_weights(pol, qp, spec)
    out, actions = _check_forward(pol, qp, spec, obs)
    # re-quantize in place (a learner broadcast) and run again: same result
    pol.quantize(layers_dev, spec.input_ranges)
    again, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK and torch.equal(again, out)
    # the scalar export refuses a per-channel layer, the per-channel export a per-tensor one
    w_q = torch.empty(spec.layers[0].weight.shape, dtype=torch.int8, device="cuda")
    with pytest.raises(B.ActorQError):
        B.actorq_policy_export_layer(pol.handle, 0, w_q)
    pol.close()


def test_debug_taps_do_not_perturb_results():
    """The debug call slows one layer's epilogue by orders of magnitude, which shifts every
    hand-off in the fused kernel's pipeline; repeated on the multi-tile 1024-wide workload, each
    run must reproduce the untapped output bit for bit (a race between the kernel's roles shows up
    here as a whole wrong tile) and leave the device status clean."""
    spec = W.build_config("mlp_wide")
    pol = B.QuantizedPolicy(spec.head, spec.obs_dtype).quantize(B.layers_to_device(spec), spec.input_ranges)
    Bsz = 65536
    obs = torch.from_numpy(W.make_obs(spec, Bsz)).cuda()
    ref, _ = pol.forward(obs)
    torch.cuda.synchronize()
    for it in range(10):
        again, _ = pol.forward(obs)
        assert torch.equal(again, ref)
        for i in range(len(spec.layers) - 1):
            n = spec.layers[i].out_features
            acc = torch.empty((Bsz, n), dtype=torch.int32, device="cuda")
            act = torch.empty((Bsz, n), dtype=torch.int8, device="cuda")
            out = torch.empty_like(ref)
            B.actorq_policy_forward_debug(pol.handle, obs, out, None, i, acc, act)
            torch.cuda.synchronize()
            assert pol.status() == B.OK, B.actorq_policy_timeout_info(pol.handle)
            assert torch.equal(out, ref), (it, i)
    pol.close()


def test_bounded_wait_reports_timeout_and_context_survives():
    """A device wait that can never be satisfied runs out after its limit, raises TIMEOUT in the
    status word, names itself in the report, and leaves the policy usable (no trap, no hang)."""
    spec = W.calibrate(W.mlp_policy("t", [8, 32, 4], seed=2), 64, seed=2)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, 50)
    before, _ = pol.forward(torch.from_numpy(obs).cuda())
    B.actorq_selftest_bounded_wait(pol.handle, 2_000_000)        # 2 ms
    torch.cuda.synchronize()
    assert pol.status() == B.ERR_TIMEOUT
    info = B.actorq_policy_timeout_info(pol.handle)
    assert info["reported"] and info["block"] == 0 and info["warp"] == 0 and info["parity"] == 0
    assert pol.status() == B.OK and not B.actorq_policy_timeout_info(pol.handle)["reported"]
    after, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert torch.equal(before, after) and pol.status() == B.OK
    _check_forward(pol, qp, spec, obs)
    pol.close()


@pytest.mark.parametrize("dims,Bsz", [([24, 256, 256, 256, 6], 300), ([128, 1024, 1024, 12], 513), ([10, 2048, 2048, 2048, 4], 70)])
def test_exploration_noise_head(dims, Bsz):
    """actorq_policy_forward_explore against the checker: tanh output, plus sigma[row] * noise, clipped.
    The 2048-wide case (the paper's ActorQ policy shape) runs on the layer-at-a-time kernels, where the
    noise is applied by a separate kernel; the others in the fused kernel's head."""
    spec = W.calibrate(W.mlp_policy("e", dims, seed=61, head="tanh"), 64, seed=61)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, Bsz, seed=61)
    rng = np.random.default_rng(61)
    sigma = rng.uniform(0.0, 0.2, Bsz).astype(np.float32)         # per actor, as in the paper's set-up
    eps = rng.standard_normal((Bsz, dims[-1])).astype(np.float32)
    eps[0] *= 100.0                                               # a row that clips
    sigma[0] = 0.2
    out = torch.empty((Bsz, dims[-1]), dtype=torch.float32, device="cuda")
    B.actorq_policy_forward_explore(pol.handle, torch.from_numpy(obs).cuda(), torch.from_numpy(sigma).cuda(),
                                    torch.from_numpy(eps).cuda(), out)
    plain, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    y_ref, _, _ = O.forward(qp, obs)
    want = O.explore(y_ref, sigma, eps)
    got = out.cpu().numpy()
    # the tanh may differ from the checker's by 1e-5 relative; the two operations after it add one ulp each
    tol = REL_TOL * np.abs(y_ref) + 2.0 ** -22
    assert np.all(np.abs(got - want) <= tol), np.abs(got - want).max()
    assert np.array_equal(got, O.explore(plain.cpu().numpy(), sigma, eps))     # exactly the library's own tanh, then the noise
    assert np.abs(got[0]).max() == 1.0
    pol.close()


def test_exploration_noise_rejects_q_value_heads():
    spec = W.calibrate(W.mlp_policy("q", [24, 64, 5], seed=62, head="linear"), 32, seed=62)
    pol, _, _ = _quantize_both(spec)
    z = torch.zeros((4, 5), device="cuda")
    with pytest.raises(B.ActorQError):
        B.actorq_policy_forward_explore(pol.handle, torch.zeros((4, 24), device="cuda"), torch.zeros(4, device="cuda"), z, z.clone())
    pol.close()


@pytest.mark.parametrize("dims,head", [([67, 2048, 2048, 21], "tanh"), ([10, 1040, 4096, 48, 5], "linear")])
def test_wide_fc_policies_run_on_the_layer_kernel(dims, head):
    """Policies wider than the fused MLP kernels take (the paper's ActorQ policies have 2048-wide
    hidden layers) run layer by layer on the tensor-core layer kernel: every layer's accumulators and
    codes, and the outputs, against the checker; observation widths that are not multiples of 16."""
    spec = W.calibrate(W.mlp_policy("wide", dims, seed=71, head=head, nonzero_bias=True), 64, seed=71)
    pol, qp, _ = _quantize_both(spec)
    with pytest.raises(B.ActorQError):
        B.actorq_policy_set_fused_variant(pol.handle, 2)          # not a fused-kernel policy
    _check_weights(pol, qp, spec)
    _check_forward(pol, qp, spec, W.make_obs(spec, 257, seed=71))
    assert B.actorq_policy_last_launch_count(pol.handle) == len(dims)      # input quantizer + one launch per layer
    pol.close()


@pytest.mark.parametrize("dims,head,Bsz", [([128, 1024, 1024, 1024, 32], "tanh", 1300),     # 6 tile pairs, the last one half empty
                                           ([40, 640, 520, 7], "argmax", 3),                # a handful of rows, greedy head
                                           ([33, 1024, 96, 12], "linear", 769)])            # 4 tile pairs, the odd tile of the last one missing
def test_policies_wider_than_512_default_to_the_layer_kernel(dims, head, Bsz):
    """A policy the fused kernels could take but with a hidden layer wider than 512 runs on the layer
    kernel unless a fused kernel is pinned: launch count = input quantizer + one launch per layer; every
    layer's accumulators and codes and the outputs against the checker (successive layers walk the
    tile pairs in opposite directions: odd and even tile-pair counts, ragged last tiles); and the pinned
    fused kernel gives the same outputs bit for bit."""
    spec = W.calibrate(W.mlp_policy("w", dims, seed=91, head=head, nonzero_bias=True), 64, seed=91)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, Bsz, seed=91)
    out, act = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    assert B.actorq_policy_last_launch_count(pol.handle) == len(dims)
    _check_forward(pol, qp, spec, obs)
    B.actorq_policy_set_fused_variant(pol.handle, 2)
    other, other_act = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    assert B.actorq_policy_last_launch_count(pol.handle) == 1
    assert torch.equal(out, other)
    if head == "argmax":
        assert torch.equal(act, other_act)
    pol.close()


@pytest.mark.parametrize("dims,head,Bsz", [([24, 256, 256, 256, 6], "tanh", 200),
                                           ([50, 416, 300, 160, 9], "linear", 700),      # chunk halves that straddle weight tiles
                                           ([33, 96, 520, 1000, 40, 3], "tanh", 385),    # narrow, ragged and 5 layers
                                           ([128, 1024, 1024, 12], "argmax", 513),
                                           ([67, 2048, 2048, 21], "tanh", 1100),         # several items per CTA pair and layer
                                           ([9, 2600, 40, 128], "linear", 257),          # 11 column chunks, the widest head
                                           ([16, 8192, 4100, 8], "tanh", 130),           # the widest hidden layer the path takes
                                           ([3, 16, 2], "tanh", 1)])
def test_layer_at_a_time_pair_kernel_matches_checker(dims, head, Bsz):
    """One launch per layer on CTA pairs (variant 3, the default of policies wider than 1024): the
    accumulators and codes of every layer and the outputs against the checker; where a fused kernel
    takes the policy too, its outputs bit for bit."""
    spec = W.calibrate(W.mlp_policy("lp", dims, seed=91, head=head, nonzero_bias=(len(dims) % 2 == 1)), 128, seed=91)
    pol, qp, _ = _quantize_both(spec)
    B.actorq_policy_set_fused_variant(pol.handle, 3)
    obs = W.make_obs(spec, Bsz, seed=91)
    out, act = _check_forward(pol, qp, spec, obs)
    assert B.actorq_policy_last_launch_count(pol.handle) == len(dims)      # input quantizer + one launch per layer
    # a second call on the same policy (row-sum counters and buffers reused) and a smaller batch after it
    again, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert torch.equal(out, again)
    if Bsz > 130:
        _check_forward(pol, qp, spec, obs[:130], check_layers=False)
    if max(dims[1:-1]) <= 1024:
        B.actorq_policy_set_fused_variant(pol.handle, 0)
        other, oact = pol.forward(torch.from_numpy(obs).cuda())
        torch.cuda.synchronize()
        assert pol.status() == B.OK
        assert torch.equal(out, other)
        if head == "argmax":
            assert torch.equal(act, oact)
    pol.close()


@pytest.mark.parametrize("dims,head,Bsz", [([20] + [64] * 15 + [4], "tanh", 130),            # 16 layers, the most a policy may have
                                           ([1024, 96, 128], "linear", 259),                    # widest observation and head the fused kernels take
                                           ([7, 1024, 1024, 1024, 1024, 1024, 128], "argmax", 3),  # deep and wide, a handful of rows
                                           ([3, 16, 2], "tanh", 1)])                            # the smallest shapes, one observation
def test_shape_extremes_of_the_fused_kernels(dims, head, Bsz):
    spec = W.calibrate(W.mlp_policy("x", dims, seed=81, head=head, nonzero_bias=True), 64, seed=81)
    pol, qp, _ = _quantize_both(spec)
    for variant in (2, 1):
        B.actorq_policy_set_fused_variant(pol.handle, variant)
        _check_forward(pol, qp, spec, W.make_obs(spec, Bsz, seed=81), check_layers=(variant == 2))
    pol.close()


@pytest.mark.parametrize("kind", ["conv", "wide_mlp", "mlp"])
def test_forward_orders_after_the_kernel_that_produces_its_input(kind):
    """The layer kernels are launched as programmatic dependents (their set-up may overlap the tail
    of the kernel before them on the stream): a forward enqueued right behind a kernel that writes
    its observations, and a second forward right behind the first on other observations, must see
    exactly those observations.  No synchronisation between the launches."""
    if kind == "conv":
        spec = W.calibrate(W.dqn_policy("pd", in_hw=(44, 44), channels=(4, 16, 32, 32), fc_hidden=64, n_actions=6), 16)
        rows = 700
    elif kind == "wide_mlp":
        spec = W.calibrate(W.mlp_policy("pd", [40, 1100, 1100, 9], seed=61, head="tanh"), 64, seed=61)
        rows = 3000
    else:
        spec = W.calibrate(W.mlp_policy("pd", [40, 256, 256, 9], seed=61, head="tanh"), 64, seed=61)
        rows = 3000
    pol, qp, layers_dev = _quantize_both(spec)
    a = torch.from_numpy(W.make_obs(spec, rows, seed=1)).cuda()
    b = torch.from_numpy(W.make_obs(spec, rows, seed=2)).cuda()
    ref_a, _ = pol.forward(a)
    ref_b, _ = pol.forward(b)
    torch.cuda.synchronize()
    ref_a, ref_b = ref_a.clone(), ref_b.clone()
    for _ in range(20):
        staged = torch.zeros_like(a)
        out_a = torch.empty_like(ref_a)
        out_b = torch.empty_like(ref_b)
        act = torch.empty((rows,), dtype=torch.int32, device="cuda") if spec.head == "argmax" else None
        act2 = torch.empty((rows,), dtype=torch.int32, device="cuda") if spec.head == "argmax" else None
        big = torch.empty((1 << 26,), dtype=torch.float32, device="cuda")
        big.fill_(1.0)                              # a long kernel in front
        staged.copy_(a)                             # the producer of the observations
        pol.forward(staged, out_a, act)
        pol.quantize(layers_dev, spec.input_ranges)  # a broadcast between two forwards (same weights)
        pol.forward(b, out_b, act2)
        torch.cuda.synchronize()
        assert pol.status() == B.OK
        assert torch.equal(out_a, ref_a) and torch.equal(out_b, ref_b)
    pol.close()


def _edge_and_random_rows(Bsz, n_random, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([np.arange(0, 130), np.arange(Bsz - 130, Bsz), rng.integers(0, Bsz, n_random)]))


@pytest.mark.parametrize("per_channel", [False, True])
@pytest.mark.parametrize("Bsz", [8192, 65536])
def test_layer_pair_kernel_many_items_per_cta_pair(per_channel, Bsz):
    """The paper's 2048-wide actor shape at batch sizes where every CTA pair of the layer kernel works
    through many (tile pair, chunk) items in a row -- 3.5 per pair at 8192 rows, 28 at 65536 -- so the
    alternating accumulators, the ring's phase wrap across items and the one-item-ahead prefetch of
    row sums and column constants all run: sampled rows (first and last 130 plus random ones)
    against the checker, every layer's accumulators and codes at 8192 rows."""
    dims = [67, 2048, 2048, 21] if per_channel else [67, 2048, 2048, 2048, 21]
    spec = W.mlp_policy("steady", dims, seed=73, head="tanh", nonzero_bias=True)
    if per_channel:
        for l in spec.layers:
            l.weight *= np.linspace(0.2, 2.0, l.weight.shape[0], dtype=np.float32).reshape(-1, 1)
            l.per_channel = True
    W.calibrate(spec, 64, seed=73)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, Bsz, seed=73)
    out, _ = _check_forward(pol, qp, spec, obs, _edge_and_random_rows(Bsz, 256, 73), check_layers=(Bsz == 8192))
    again, _ = pol.forward(torch.from_numpy(obs).cuda())        # buffers and row-sum counters reused
    torch.cuda.synchronize()
    assert pol.status() == B.OK and torch.equal(out, again)
    pol.close()


@pytest.mark.parametrize("config,Bsz", [("mlp_wide", 65536), ("d4pg_humanoid", 40000)])
def test_single_cta_fused_kernel_many_tiles_per_cta(config, Bsz):
    """The single-CTA fused kernel with several tiles per CTA (512 and 313 tiles on 148 CTAs): its
    persistent tile loop, the double-buffered first operand and the per-tile row sums, sampled rows
    against the checker, and the whole batch bit for bit against the CTA-pair kernel."""
    spec = W.build_config(config)
    pol, qp, _ = _quantize_both(spec)
    B.actorq_policy_set_fused_variant(pol.handle, 1)
    obs = W.make_obs(spec, Bsz, seed=7)
    out, _ = _check_forward(pol, qp, spec, obs, _edge_and_random_rows(Bsz, 256, 7), check_layers=True)
    B.actorq_policy_set_fused_variant(pol.handle, 2)
    other, _ = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK and torch.equal(out, other)
    pol.close()


@pytest.mark.parametrize("dims,head,Bsz", [([67, 256, 256, 256, 21], "tanh", 80000),       # five tile pairs per CTA pair: both slots, odd count
                                           ([24, 256, 256, 256, 6], "tanh", 40000),        # even head width, 16-byte-aligned rows
                                           ([67, 256, 256, 256, 21], "tanh", 37888 + 129),  # ragged last tile read from global memory
                                           ([50, 200, 96, 160, 9], "argmax", 20000),       # ragged widths, greedy actions
                                           ([33, 64, 256, 40, 3], "linear", 777),
                                           ([20] + [64] * 15 + [4], "tanh", 300),           # 16 layers
                                           ([3, 4], "linear", 5)])                         # a single layer: the head alone
def test_resident_weights_kernel_matches_checker(dims, head, Bsz):
    """The small-policy kernel (all int8 weights resident in shared memory, observation tiles staged
    by bulk copies, two tiles in flight per CTA): every layer's accumulators and codes and the outputs
    on sampled rows against the checker, and the whole batch bit for bit against the streaming
    CTA-pair kernel."""
    spec = W.calibrate(W.mlp_policy("r", dims, seed=41, head=head, nonzero_bias=(len(dims) % 2 == 0)), 128, seed=41)
    pol, qp, _ = _quantize_both(spec)
    B.actorq_policy_set_fused_variant(pol.handle, 4)
    obs = W.make_obs(spec, Bsz, seed=41)
    sample = None if Bsz <= 1000 else _edge_and_random_rows(Bsz, 256, 41)
    out, act = _check_forward(pol, qp, spec, obs, sample)
    assert B.actorq_policy_last_launch_count(pol.handle) == 1
    B.actorq_policy_set_fused_variant(pol.handle, 2)
    other, oact = pol.forward(torch.from_numpy(obs).cuda())
    torch.cuda.synchronize()
    assert pol.status() == B.OK and torch.equal(out, other)
    if act is not None:
        assert torch.equal(act, oact)
    # an observation tensor that is only 4-byte aligned is rejected by the API, one that is 16-byte aligned
    # but offset from the allocation start is fine
    B.actorq_policy_set_fused_variant(pol.handle, 4)
    if Bsz > 300:
        shifted = torch.from_numpy(obs).cuda()[4:]
        out2, _ = pol.forward(shifted.contiguous() if (shifted.data_ptr() & 15) else shifted)
        torch.cuda.synchronize()
        assert torch.equal(out2, out[4:])
    pol.close()


@pytest.mark.parametrize("dims,Bsz", [([67, 256, 256, 256, 21], 3000), ([24, 256, 256, 256, 6], 130),   # drawn in the resident kernel's head
                                      ([128, 1024, 1024, 12], 513), ([10, 2048, 2048, 4], 70)])          # drawn by the kernel behind the forward
def test_seeded_exploration_noise(dims, Bsz):
    """actorq_policy_forward_explore_seeded against the checker's Philox-4x32-10 + Box-Muller draws.  The
    integer part of the generator is exact on both sides; the normal transform runs in single precision on
    the GPU (logarithm, square root, sine / cosine: a few ulp each, |z| <= 5.7) and in double in the checker,
    so sigma * z may differ by 0.2 * 5.7 * 1e-6; on top of that the 1e-5 relative tolerance of tanh."""
    spec = W.calibrate(W.mlp_policy("es", dims, seed=63, head="tanh"), 64, seed=63)
    pol, qp, _ = _quantize_both(spec)
    obs = W.make_obs(spec, Bsz, seed=63)
    sigma = np.random.default_rng(63).uniform(0.0, 0.2, Bsz).astype(np.float32)
    sigma[0] = 0.0
    seed, first_row = 0x1234_5678_9ABC_DEF0, 2 ** 32 - 7                   # rows straddle the second counter word
    out = torch.empty((Bsz, dims[-1]), dtype=torch.float32, device="cuda")
    obs_d, sigma_d = torch.from_numpy(obs).cuda(), torch.from_numpy(sigma).cuda()
    B.actorq_policy_forward_explore_seeded(pol.handle, obs_d, sigma_d, seed, out, first_row=first_row)
    plain, _ = pol.forward(obs_d)
    torch.cuda.synchronize()
    assert pol.status() == B.OK
    y_ref, _, _ = O.forward(qp, obs)
    want = O.explore_seeded(y_ref, sigma, seed, row0=first_row)
    got = out.cpu().numpy()
    tol = REL_TOL * np.abs(y_ref) + 2.0e-6
    assert np.all(np.abs(got - want) <= tol), float(np.abs(got - want).max())
    assert np.array_equal(got[0], plain.cpu().numpy()[0])                  # sigma 0: the policy's own action
    assert np.abs(got - plain.cpu().numpy()).max() > 0.05                  # and the noise is really there
    # a row's noise does not depend on the batch: the second half alone, with its own first row
    h = Bsz // 2
    out2 = torch.empty((Bsz - h, dims[-1]), dtype=torch.float32, device="cuda")
    B.actorq_policy_forward_explore_seeded(pol.handle, obs_d[h:].clone(), sigma_d[h:].clone(), seed, out2, first_row=first_row + h)
    torch.cuda.synchronize()
    assert torch.equal(out2, out[h:])
    pol.close()
