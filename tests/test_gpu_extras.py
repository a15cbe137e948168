"""GPU parity of the outputs beyond logits / action / log-prob: the state value V(s) and the
entropy of the action distribution (Section 2.2, Eq. KD; Section 2.3, Eq. V-trace), the Monitor's KL
indicators (Section 2.4, Eq. KL), the V-trace targets (Eq. V-trace) and the per-state mixing of two
policies (Section 3.2) -- each against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
import workloads as W
from parity_util import ATOL, RTOL, compare

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _policy(name, layers=None, rows=64, seed=77):
    c = W.config(name)
    layers = W.with_value_head(c["layers"]) if layers is None else layers
    return oracle.calibrate(c["in_kind"], c["in_shape"], layers, W.parameters_for(layers, seed),
                            W.calibration_batch(name, rows), c["prune24"])


def _run(pol, obs, u, flags=0):
    import paper_2211_15023_b200 as P
    g = P.Policy(pol, obs.shape[0], flags=flags)
    out = {k: v.cpu().numpy() for k, v in g.act_ex(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda()).items()}
    g.check()
    plan = g.info()["plan"]
    g.close()
    return out, plan


@pytest.mark.parametrize("name,b", [("cartpole_mlp", 160), ("lunarlander_mlp", 517), ("nature_cnn_b160", 37),
                                    ("student_cnn_b8192", 300), ("impala_resnet_b16384", 9)])
@pytest.mark.parametrize("flags", [0, 2], ids=["production_plan", "generic_plan"])
def test_value_and_entropy_match_the_oracle(name, b, flags):
    """A value column on the last layer and the entropy, on every kind of plan: the single-launch
    MLP, the last layer fused with the sampler, and the CUDA-core kernels with a sampler launch
    of their own.  V is compared bit for bit (one fma of the same integers), H at the log-prob
    tolerance; everything else must be what the policy without the extras gives."""
    pol = _policy(name)
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(pol, obs, u, keep=False)
    out, plan = _run(pol, obs, u, flags)
    assert out["logits"].shape == (b, W.n_actions(name))
    compare(ref, out["logits"], out["actions"], out["logp"], value=out["value"], entropy=out["entropy"])
    if flags == 0 and name != "impala_resnet_b16384":
        assert "mlp_fused_kernel" in plan or "fc_sample_kernel" in plan, plan


def test_value_and_entropy_with_more_than_32_actions():
    """40 actions + V: the tensor-core kernel writes rows of 41 floats into the handle's scratch
    and the wide sampler splits them."""
    layers = W.with_value_head(W.nature_cnn(16, 32, 32, 256, actions=40))
    pol = _policy("student_cnn_b8192", layers)
    b = 45
    obs, u = W.observations("student_cnn_b8192", b), W.uniforms("student_cnn_b8192", b)
    ref = oracle.forward(pol, obs, u, keep=False)
    out, plan = _run(pol, obs, u)
    assert "sample_wide_kernel" in plan and "tc_gemm_kernel" in plan, plan
    compare(ref, out["logits"], out["actions"], out["logp"], value=out["value"], entropy=out["entropy"])


def test_entropy_without_a_value_head_and_refusal_of_a_value_pointer():
    import paper_2211_15023_b200 as P
    name, b = "nature_cnn_b160", 50
    c = W.config(name)
    pol = _policy(name, c["layers"])
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(pol, obs, u, keep=False)
    out, _ = _run(pol, obs, u)
    assert "value" not in out
    compare(ref, out["logits"], out["actions"], out["logp"], entropy=out["entropy"])
    g = P.Policy(pol, b)
    o, uu = torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda()
    t = g.act(o, uu)
    v = torch.empty(b, device="cuda")
    st = P.library().accerl_policy_act_ex(g._h, o.data_ptr(), uu.data_ptr(), b, t[0].data_ptr(), t[1].data_ptr(),
                                          t[2].data_ptr(), v.data_ptr(), None, 0)
    assert st == 1 and b"VALUE_HEAD" in P.library().accerl_last_error()
    g.close()


@pytest.mark.parametrize("b,a", [(1, 2), (777, 18), (300, 40), (5, 1)])
def test_kl_indicators(b, a):
    import paper_2211_15023_b200 as P
    rng = np.random.default_rng(b * 100 + a)
    zo = (rng.standard_normal((b, a)) * 3).astype(np.float32)
    zs = (zo + rng.standard_normal((b, a)) * rng.choice([1e-3, 0.5, 4.0], size=(b, 1))).astype(np.float32)
    zs[0] = zo[0]  # identical rows: KL = 0
    want = oracle.kl(zo, zs)
    kl, stats = P.kl(torch.from_numpy(zo).cuda(), torch.from_numpy(zs).cuda())
    kl, stats = kl.cpu().numpy(), stats.cpu().numpy()
    np.testing.assert_allclose(kl, want, rtol=RTOL, atol=ATOL)
    assert kl[0] == 0.0
    np.testing.assert_allclose(stats[0], want.mean(), rtol=RTOL, atol=ATOL)
    np.testing.assert_allclose(stats[1], want.max(), rtol=RTOL, atol=ATOL)


@pytest.mark.parametrize("n,b", [(16, 8192), (5, 160), (1, 3), (37, 1001)])
@pytest.mark.parametrize("with_discounts", [False, True])
def test_vtrace_matches_the_definition(n, b, with_discounts):
    import paper_2211_15023_b200 as P
    r = W.rollouts(n, b, seed=n * 1000 + b)
    disc = r["discounts"] if with_discounts else None
    for rho_hat, c_hat in ((1.0, 1.0), (2.0, 0.5)):
        want = oracle.vtrace(r["logp_smaller"], r["logp_original"], r["rewards"], r["values"], r["bootstrap"],
                             r["gamma"], rho_hat, c_hat, disc)
        cu = lambda k: torch.from_numpy(r[k]).cuda()  # noqa: E731
        vs, adv = P.vtrace(cu("logp_smaller"), cu("logp_original"), cu("rewards"), cu("values"), cu("bootstrap"),
                           r["gamma"], rho_hat, c_hat, None if disc is None else torch.from_numpy(disc).cuda())
        np.testing.assert_allclose(vs.cpu().numpy(), want["vs"], rtol=RTOL, atol=ATOL)
        np.testing.assert_allclose(adv.cpu().numpy(), want["adv"], rtol=RTOL, atol=ATOL)


def test_vtrace_rejects_bad_arguments():
    import paper_2211_15023_b200 as P
    lib = P.library()
    x = torch.zeros(8, device="cuda")
    p = x.data_ptr()
    assert lib.accerl_vtrace(p, p, p, p, p, None, 0, 4, 0.99, 1.0, 1.0, p, None, 0) == 1
    assert lib.accerl_vtrace(p, p, p, p, p, None, 2, 4, 0.99, 0.0, 1.0, p, None, 0) == 1
    assert lib.accerl_vtrace(None, p, p, p, p, None, 2, 4, 0.99, 1.0, 1.0, p, None, 0) == 1
    assert lib.accerl_vtrace(p, p, p, p, p, None, 2, 4, 0.99, 1.0, 1.0, p + 2, None, 0) == 1


@pytest.mark.parametrize("alpha", [0.0, 0.3, 1.0])
def test_mixing_of_two_policies(alpha):
    """Student and original Nature-CNN (both with a value head) on the same states: every state's
    outputs are those of the network its selector draw picks."""
    import paper_2211_15023_b200 as P
    b = 203
    small = _policy("student_cnn_b8192", seed=5)
    orig = _policy("nature_cnn_b160", seed=6)
    obs, u = W.observations("nature_cnn_b160", b), W.uniforms("nature_cnn_b160", b)
    usel = np.random.default_rng(9).random(b, dtype=np.float32)
    ref = oracle.forward_mixed(small, orig, obs, u, usel, alpha)
    gs, go = P.Policy(small, b), P.Policy(orig, b)
    for _ in range(2):  # the second call reuses the buffers the first one allocated
        out = {k: v.cpu().numpy() for k, v in
               P.act_mixed(gs, go, torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda(),
                           torch.from_numpy(usel).cuda(), alpha).items()}
        gs.check()
        go.check()
        assert np.array_equal(out["use_smaller"].astype(bool), ref["use_smaller"])
        compare(ref, out["logits"], out["actions"], out["logp"], value=out["value"], entropy=out["entropy"])
    if 0.0 < alpha < 1.0:
        assert 0 < out["use_smaller"].sum() < b
    gs.close()
    go.close()


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_handle_usable():
    """The give-up path of the bounded waits: a one-warp kernel waits, with a limit of a few hundred
    polls, on a barrier nothing arrives at; the status word is set, check() reports TIMEOUT once,
    and the next step runs and checks clean."""
    import paper_2211_15023_b200 as P
    name, b = "nature_cnn_b160", 16
    pol = W.drawn_int8_policy(name)
    g = P.Policy(pol, b)
    obs, u = torch.from_numpy(W.observations(name, b)).cuda(), torch.from_numpy(W.uniforms(name, b)).cuda()
    first = [t.clone() for t in g.act(obs, u)]
    g.check()
    g.selftest_wait(300)
    with pytest.raises(P.AccerlError) as e:
        g.check()
    assert e.value.status == 6 and "0x80" in str(e.value)
    g.check()  # the word was cleared
    again = g.act(obs, u)
    g.check()
    for x, y in zip(first, again):
        assert torch.equal(x, y)
    g.close()


@pytest.mark.parametrize("name,rows", [("cartpole_mlp", 256), ("lunarlander_mlp", 300), ("nature_cnn_b160", 48),
                                       ("student_cnn_b8192", 40), ("impala_resnet_b16384", 12)])
def test_quantisation_and_calibration_on_the_device(name, rows):
    """accerl_policy_create_fp32 against the oracle's quantiser and calibrator: int8 weights (2:4
    pruned for the residual network), weight scales, every activation scale and the residual
    multipliers must be the same bits, and the policy built from them must act like the oracle's."""
    import paper_2211_15023_b200 as P
    c = W.config(name)
    params = W.fp32_parameters(name)
    calib = W.calibration_batch(name, rows)
    want = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], params, calib, c["prune24"])
    b = 19
    g = P.Policy.from_fp32(c["in_kind"], c["in_shape"], c["layers"], params, calib, b, prune24=c["prune24"])
    for i, l in enumerate(want["layers"]):
        got = g.export(i)
        assert got["s_in"] == np.float32(l["s_in"]) and got["s_out"] == np.float32(l["s_out"]), (i, got["s_in"], l["s_in"], got["s_out"], l["s_out"])
        if l["kind"] == "maxpool":
            continue
        assert np.array_equal(got["w"], l["w"]), "layer %d: int8 weights differ" % i
        assert np.array_equal(got["s_w"], l["s_w"]), "layer %d: weight scales differ" % i
        if l["skip_from"] >= 0:
            assert np.array_equal(got["skip_mul"], l["skip_mul"]), "layer %d: residual multipliers differ" % i
        if c["prune24"]:
            k = got["w"].transpose(0, 2, 3, 1).reshape(got["w"].shape[0], -1, 4)
            assert ((k != 0).sum(-1) <= 2).all()
    obs, u = W.observations(name, b), W.uniforms(name, b)
    ref = oracle.forward(want, obs, u, keep=False)
    out = [t.cpu().numpy() for t in g.act(torch.from_numpy(obs).cuda(), torch.from_numpy(u).cuda())]
    g.check()
    compare(ref, *out)
    g.close()


def test_tensor_pipe_probe_reports_plausible_costs_and_rejects_bad_arguments():
    """accerl_tc_probe_i8: an N = 256 MMA is bound by its multiply-accumulates (8192 per cycle and
    SM: 128 cycles), a narrow one by reading its operands from shared memory (about 40 cycles);
    layout and row shift of the operands must not matter; bad arguments are refused on the host."""
    import paper_2211_15023_b200 as P
    wide = P.tc_probe_i8(256, 2, 2048, 148)
    assert 120 <= wide["cycles_per_mma"] <= 140 and wide["tops"] > 3000, wide
    narrow = P.tc_probe_i8(32, 1, 2048, 148)
    assert 35 <= narrow["cycles_per_mma"] <= 50, narrow
    shifted = P.tc_probe_i8(32, 1, 2048, 8, 64, 21, 8)
    assert abs(shifted["cycles_per_mma"] - narrow["cycles_per_mma"]) < 3, (shifted, narrow)
    for bad in ((24, 1, 2048, 1), (256, 4, 2048, 1), (32, 1, 2050, 1), (32, 5, 2048, 1), (32, 1, 2048, 1, 48)):
        with pytest.raises(P.AccerlError) as e:
            P.tc_probe_i8(*bad)
        assert e.value.status == 1
