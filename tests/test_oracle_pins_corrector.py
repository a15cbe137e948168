"""Pins for the oracle's value head, entropy, KL and V-trace functions (no GPU needed).

Each is checked against something that is not the oracle: hand-worked fixtures, closed forms,
scipy routines, the n-step return and the one-step TD target, and brute force on tiny inputs.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
import workloads as W
from test_oracle_pins import _parse_worked, _worked_policy

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line)
    return out


# --------------------------------------------------------------------------
# value head and entropy
# --------------------------------------------------------------------------

def test_worked_example_value_head_and_entropy():
    v, rows = _parse_worked()
    lines = _rows("worked_example_value_entropy.txt")
    extra = {l.split(" ", 1)[0]: np.array([float(t) for t in l.split(" ", 1)[1].split()])
             for l in lines if not l.startswith("row")}
    gold = [[[float(t) for t in part.split()] for part in l[4:].split("|")]
            for l in lines if l.startswith("row")]
    pol = _worked_policy(v)
    last = pol["layers"][-1]
    last["w"] = np.concatenate([last["w"], extra["w_v"].astype(np.int8).reshape(1, 3, 1, 1)])
    last["s_w"] = np.concatenate([last["s_w"], extra["s_w_v"].astype(np.float32)])
    last["bias"] = np.concatenate([last["bias"], extra["b_v"].astype(np.float32)])
    last["out_c"], last["value"] = 3, True
    assert len(gold) == len(rows)
    for (obs, q_in, acc1, q1, acc2, logits, logp, ua), (gq1, gacc, gval, gent) in zip(rows, gold):
        assert q1 == gq1
        r = oracle.forward(pol, np.array([obs], np.float32), np.array([ua[0]], np.float32))
        assert r["logits"].shape == (1, 2) and r["logits"].ravel().tolist() == logits
        assert r["value"].tolist() == gval                     # exact: dyadic arithmetic
        assert int(r["actions"][0]) == int(ua[1])              # the value column is no action
        np.testing.assert_allclose(r["entropy"], gent, atol=1e-11, rtol=0)


def test_entropy_closed_forms_and_library():
    for a in (1, 2, 3, 18, 40):
        h = oracle.entropy(np.full((1, a), 3.25, np.float32))
        np.testing.assert_allclose(h, math.log(a), atol=1e-14)         # uniform: log A
    # one-hot limit: one logit far above the rest -> 0 (and never negative or NaN)
    z = np.zeros((1, 18), np.float32)
    z[0, 5] = 200.0
    h = oracle.entropy(z)
    assert 0.0 <= h[0] < 1e-80
    # two actions: H = -p log p - (1-p) log(1-p) with p = sigmoid(z0 - z1)
    for d in (-7.5, -1.0, 0.25, 3.0, 20.0):
        p = 1.0 / (1.0 + math.exp(-d))
        want = -(p * math.log(p) + (1 - p) * math.log1p(-p))
        np.testing.assert_allclose(oracle.entropy(np.array([[d, 0.0]], np.float32)), want, rtol=1e-12,
                                   atol=1e-14)
    rng = np.random.default_rng(3)
    z = (rng.standard_normal((64, 18)) * 4).astype(np.float32)
    want = scipy.stats.entropy(scipy.special.softmax(z.astype(np.float64), axis=1), axis=1)
    np.testing.assert_allclose(oracle.entropy(z), want, rtol=1e-12)
    np.testing.assert_allclose(oracle.entropy(z + np.float32(8.0)), oracle.entropy(z), rtol=1e-5)


def test_kl_closed_forms_and_library():
    rng = np.random.default_rng(4)
    zo = (rng.standard_normal((50, 18)) * 3).astype(np.float32)
    zs = (rng.standard_normal((50, 18)) * 3).astype(np.float32)
    assert np.all(np.abs(oracle.kl(zo, zo)) < 1e-15)                     # KL(p || p) = 0
    po, ps = (scipy.special.softmax(z.astype(np.float64), axis=1) for z in (zo, zs))
    want = scipy.special.rel_entr(po, ps).sum(axis=1)
    got = oracle.kl(zo, zs)
    np.testing.assert_allclose(got, want, rtol=1e-11)
    assert np.all(got >= 0)
    # the direction matters: the expectation is under pi_original (first argument)
    p, q = np.array([0.9, 0.1]), np.array([0.5, 0.5])
    lo, ls = np.log(p)[None].astype(np.float32), np.log(q)[None].astype(np.float32)
    np.testing.assert_allclose(oracle.kl(lo, ls), 0.9 * math.log(1.8) + 0.1 * math.log(0.2), rtol=1e-6)
    np.testing.assert_allclose(oracle.kl(ls, lo), 0.5 * math.log(1 / 1.8) + 0.5 * math.log(5.0), rtol=1e-6)
    # an action pi_original never takes contributes nothing, however unlikely under pi_smaller
    lo = np.array([[0.0, -300.0]], np.float32)
    ls = np.array([[0.0, 0.0]], np.float32)
    np.testing.assert_allclose(oracle.kl(lo, ls), math.log(2.0), rtol=1e-12)


def test_forward_mixed_selects_per_state():
    name = "cartpole_mlp"
    c = W.config(name)
    small = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                             W.calibration_batch(name, 64))
    orig = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name, seed=77),
                            W.calibration_batch(name, 64))
    obs, u = W.observations(name, 40), W.uniforms(name, 40)
    sel = np.linspace(0, 1, 40, endpoint=False).astype(np.float32)
    rs, ro = oracle.forward(small, obs, u, keep=False), oracle.forward(orig, obs, u, keep=False)
    for alpha in (0.0, 0.3, 1.0):
        m = oracle.forward_mixed(small, orig, obs, u, sel, alpha)
        pick = sel < np.float32(alpha)
        assert pick.sum() == round(alpha * 40) and np.array_equal(m["use_smaller"], pick)
        assert np.array_equal(m["logits"][pick], rs["logits"][pick])
        assert np.array_equal(m["logits"][~pick], ro["logits"][~pick])
        assert np.array_equal(m["actions"], np.where(pick, rs["actions"], ro["actions"]))
        assert np.array_equal(m["logp"], np.where(pick, rs["logp"], ro["logp"]))


# --------------------------------------------------------------------------
# V-trace
# --------------------------------------------------------------------------

def _nums(s):
    return np.array([float(t) for t in s.split()], np.float64)


def test_vtrace_hand_worked_rollouts():
    cases = [l[5:] for l in _rows("vtrace_3step.txt") if l.startswith("case ")]
    assert len(cases) == 3
    for line in cases:
        head, ps, po, r, v, boot, disc, vs, adv = [t.strip() for t in line.split("|")]
        gamma, rho_hat, c_hat = _nums(head)
        col = lambda a: np.asarray(a, np.float32).reshape(-1, 1)  # noqa: E731
        out = oracle.vtrace(col(np.log(_nums(ps))), col(np.log(_nums(po))), col(_nums(r)), col(_nums(v)),
                            _nums(boot).astype(np.float32), gamma, rho_hat, c_hat,
                            None if disc == "-" else col(_nums(disc)))
        np.testing.assert_allclose(out["vs"].ravel(), _nums(vs), atol=1e-6, rtol=0)
        np.testing.assert_allclose(out["adv"].ravel(), _nums(adv), atol=1e-6, rtol=0)


def _rollout(rng, n, b):
    lps = np.log(rng.uniform(0.05, 1.0, (n, b))).astype(np.float32)
    lpo = np.log(rng.uniform(0.05, 1.0, (n, b))).astype(np.float32)
    return (lps, lpo, rng.standard_normal((n, b)).astype(np.float32),
            rng.standard_normal((n, b)).astype(np.float32), rng.standard_normal(b).astype(np.float32))


def test_vtrace_on_policy_is_the_n_step_return():
    # equal policies, rho_hat = c_hat = 1: v_s = sum_{t>=s} g^(t-s) r_t + g^(n-s) V(x_n)
    rng = np.random.default_rng(8)
    n, b, g = 16, 5, float(np.float32(0.99))   # gamma crosses the C interface as fp32
    lps, _, r, v, boot = _rollout(rng, n, b)
    out = oracle.vtrace(lps, lps, r, v, boot, g)
    for s in range(n):
        want = sum(g ** (t - s) * r[t].astype(np.float64) for t in range(s, n)) + g ** (n - s) * boot.astype(np.float64)
        np.testing.assert_allclose(out["vs"][s], want, rtol=1e-9, atol=1e-9)
    # and the advantage is the n-step return from s+1 on, minus V(x_s)
    nxt = np.concatenate([out["vs"][1:], boot[None].astype(np.float64)])
    np.testing.assert_allclose(out["adv"], r + g * nxt - v, rtol=1e-9, atol=1e-9)


def test_vtrace_c_hat_zero_is_the_one_step_td_target():
    rng = np.random.default_rng(9)
    n, b, g = 5, 7, float(np.float32(0.9))
    lps, lpo, r, v, boot = _rollout(rng, n, b)
    out = oracle.vtrace(lps, lpo, r, v, boot, g, rho_hat=1.0, c_hat=0.0)
    rho = np.minimum(1.0, np.exp(lpo.astype(np.float64) - lps))
    v_next = np.concatenate([v[1:], boot[None]]).astype(np.float64)
    np.testing.assert_allclose(out["vs"], v + rho * (r + g * v_next - v), rtol=1e-12, atol=1e-12)


def test_vtrace_clipping_recursion_and_independence():
    rng = np.random.default_rng(10)
    n, b, g = 16, 9, float(np.float32(0.99))
    lps, lpo, r, v, boot = _rollout(rng, n, b)
    ratio = np.exp(lpo.astype(np.float64) - lps)
    assert (ratio > 1.5).any() and (ratio < 0.5).any()          # both sides of every clip level
    for rho_hat, c_hat in ((1.0, 1.0), (1.5, 0.5), (100.0, 100.0)):
        out = oracle.vtrace(lps, lpo, r, v, boot, g, rho_hat, c_hat)
        rho, c = np.minimum(rho_hat, ratio), np.minimum(c_hat, ratio)
        v_next = np.concatenate([v[1:], boot[None]]).astype(np.float64)
        delta = rho * (r + g * v_next - v)
        # the definition satisfies v_s - V(x_s) = delta_s + g c_s (v_{s+1} - V(x_{s+1}))
        d = out["vs"] - v
        d_next = np.concatenate([d[1:], np.zeros((1, b))])
        np.testing.assert_allclose(d, delta + g * c * d_next, rtol=1e-10, atol=1e-10)
    # trajectories do not interact, and a one-step rollout is the plain TD target
    one = oracle.vtrace(lps[:, 3:4], lpo[:, 3:4], r[:, 3:4], v[:, 3:4], boot[3:4], g)
    np.testing.assert_allclose(one["vs"], oracle.vtrace(lps, lpo, r, v, boot, g)["vs"][:, 3:4], rtol=1e-15)
    o1 = oracle.vtrace(lps[:1], lpo[:1], r[:1], v[:1], boot, g)
    np.testing.assert_allclose(o1["vs"][0], v[0] + np.minimum(1.0, ratio[0]) * (r[0] + g * boot.astype(np.float64) - v[0]),
                               rtol=1e-12)
    # per-step discounts equal to gamma everywhere change nothing; a zero cuts the sums
    same = oracle.vtrace(lps, lpo, r, v, boot, 123.0, discounts=np.full((n, b), g, np.float32))
    np.testing.assert_allclose(same["vs"], oracle.vtrace(lps, lpo, r, v, boot, np.float32(g))["vs"], rtol=1e-12)
    disc = np.full((n, b), g, np.float32)
    disc[6] = 0.0
    cut = oracle.vtrace(lps, lpo, r, v, boot, g, discounts=disc)
    head = oracle.vtrace(lps[:7], lpo[:7], r[:7], v[:7], np.zeros(b, np.float32), g, discounts=disc[:7])
    np.testing.assert_allclose(cut["vs"][:7], head["vs"], rtol=1e-12, atol=1e-12)
