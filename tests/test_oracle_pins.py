"""Pins for the CPU oracle: everything here runs without a GPU.

Each test checks the oracle against something that is not the oracle: a
hand-worked example, float64 library convolutions on integer tensors, an fp64
de-quantised forward written with a different loop structure, structural
special cases, brute force, and invariants of a probability distribution.
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

import oracle
import workloads as W
from oracle import net as ON

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# hand-worked two-layer example
# --------------------------------------------------------------------------

def _parse_worked():
    vals, rows = {}, []
    for line in open(os.path.join(GOLD, "worked_example_2layer.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(" ", 1)
        if key == "row":
            rows.append([[float(t) for t in part.split()] for part in rest.split("|")])
        elif ";" in rest:
            vals[key] = np.array([[float(t) for t in r.split()] for r in rest.split(";")])
        else:
            vals[key] = np.array([float(t) for t in rest.split()])
    return vals, rows


def _worked_policy(v):
    l1 = dict(kind="fc", in_c=2, in_h=1, in_w=1, out_c=3, kh=1, kw=1, stride=1, pad=0,
              relu_in=False, relu_out=True, logits=False, skip_from=-1, skip_mul=None,
              w=v["w1"].astype(np.int8).reshape(3, 2, 1, 1), s_w=v["s_w1"].astype(np.float32),
              bias=v["b1"].astype(np.float32), s_in=np.float32(v["s_input"][0]),
              s_out=np.float32(v["s_out1"][0]))
    l2 = dict(l1, in_c=3, out_c=2, relu_out=False, logits=True,
              w=v["w2"].astype(np.int8).reshape(2, 3, 1, 1), s_w=v["s_w2"].astype(np.float32),
              bias=v["b2"].astype(np.float32), s_in=np.float32(v["s_out1"][0]),
              s_out=np.float32(1.0))
    return dict(in_kind="f32", in_shape=(2, 1, 1), s_input=np.float32(v["s_input"][0]),
                layers=[l1, l2])


def test_worked_example_every_intermediate():
    v, rows = _parse_worked()
    pol = _worked_policy(v)
    assert len(rows) >= 5
    for obs, q_in, acc1, q1, acc2, logits, logp, ua in rows:
        o = np.array([obs], np.float32)
        q = ON.ingest("f32", o, pol["s_input"])
        assert q.ravel().tolist() == q_in
        a1 = ON.layer_acc(pol["layers"][0], q.reshape(1, 2, 1, 1))
        assert a1.ravel().tolist() == acc1
        h = ON.requant(ON.layer_float(pol["layers"][0], a1), pol["layers"][0]["s_out"])
        assert h.ravel().tolist() == q1
        a2 = ON.layer_acc(pol["layers"][1], h)
        assert a2.ravel().tolist() == acc2
        for k in range(0, len(ua), 2):
            r = oracle.forward(pol, o, np.array([ua[k]], np.float32))
            assert r["logits"].ravel().tolist() == logits  # exact: dyadic arithmetic
            np.testing.assert_allclose(r["logp_all"].ravel(), logp, atol=2e-8, rtol=0)
            assert int(r["actions"][0]) == int(ua[k + 1])
            np.testing.assert_allclose(r["logp"][0], logp[int(ua[k + 1])], atol=1e-7)


# --------------------------------------------------------------------------
# input stage
# --------------------------------------------------------------------------

def test_ingest_all_256_bytes():
    from fractions import Fraction as Fr
    s = np.float32(1.0) / np.float32(127.0)
    u = np.arange(256, dtype=np.uint8)
    q = ON.ingest("u8", u, s).astype(np.int64)
    assert q[0] == 0 and q[255] == 127
    assert np.all(np.diff(q) >= 0) and q.min() >= 0
    for b in range(256):
        exact = Fr(b, 255) / Fr(float(s))  # infinitely precise x / s
        assert abs(Fr(int(q[b])) - exact) <= Fr(1, 2) + Fr(1, 10000), b
    # a coarser scale must saturate at +127, a finer one keeps small bytes apart
    assert ON.ingest("u8", u, np.float32(1.0 / 400.0)).max() == 127
    assert ON.ingest("u8", np.array([3], np.uint8), np.float32(1.0 / 255.0))[0] == 3


def test_ingest_f32_ties_to_even_and_both_clamps():
    s = np.float32(0.25)
    obs = np.array([0.625, 0.875, -0.625, -0.875, 0.124, 100.0, -100.0, 31.875, -32.125], np.float32)
    # obs / s = 2.5, 3.5, -2.5, -3.5, 0.496, 400, -400, 127.5, -128.5
    want = [2, 4, -2, -4, 0, 127, -128, 127, -128]
    assert ON.ingest("f32", obs, s).tolist() == want


# --------------------------------------------------------------------------
# accumulators against float64 library routines on integer tensors (exact < 2^53)
# --------------------------------------------------------------------------

def _all_layer_shapes():
    seen, out = set(), []
    for name, c in W.CONFIGS.items():
        for l in c["layers"]:
            key = tuple(l[k] for k in ("kind", "in_c", "in_h", "in_w", "out_c", "kh", "stride",
                                       "pad", "relu_in"))
            if key not in seen:
                seen.add(key)
                out.append(l)
    return out


@pytest.mark.parametrize("l", _all_layer_shapes(),
                         ids=lambda l: "%s_%dx%dx%d_to_%d_k%d" % (l["kind"], l["in_c"], l["in_h"],
                                                                  l["in_w"], l["out_c"], l["kh"]))
def test_accumulators_equal_float64_library(l):
    rng = np.random.default_rng(7)
    b = 2
    x = rng.integers(-128, 128, (b, l["in_c"], l["in_h"], l["in_w"])).astype(np.int8)
    if l["kind"] == "maxpool":
        got = ON.maxpool(l, x)
        ref = TF.max_pool2d(torch.from_numpy(x.astype(np.float64)), l["kh"], l["stride"])
        assert np.array_equal(got, ref.numpy().astype(np.int8))
        return
    e = dict(l, skip_from=-1)
    e["w"] = rng.integers(-127, 128, (l["out_c"], l["in_c"], l["kh"], l["kw"])).astype(np.int8)
    acc = ON.layer_acc(e, x)
    xt = torch.from_numpy(x.astype(np.float64))
    if l["relu_in"]:
        xt = xt.clamp(min=0)
    wt = torch.from_numpy(e["w"].astype(np.float64))
    if l["kind"] == "conv":
        ref = TF.conv2d(xt, wt, stride=l["stride"], padding=l["pad"])
    else:
        ref = TF.linear(xt.reshape(b, -1), wt.reshape(l["out_c"], -1)).reshape(b, -1, 1, 1)
    assert acc.shape == tuple(ref.shape)
    assert np.array_equal(acc.astype(np.float64), ref.numpy())


def test_fc_flatten_order_is_c_h_w():
    # an fc layer fed by a conv output reads it in (C, H, W) order: weight column
    # c*H*W + y*W + x multiplies activation [c, y, x]
    rng = np.random.default_rng(3)
    x = rng.integers(-128, 128, (1, 3, 2, 5)).astype(np.int8)
    w = np.zeros((1, 30, 1, 1), np.int8)
    c, y, xx = 2, 1, 3
    w[0, c * 10 + y * 5 + xx] = 1
    l = dict(kind="fc", in_c=30, out_c=1, kh=1, kw=1, stride=1, pad=0, in_h=1, in_w=1,
             relu_in=False, skip_from=-1, w=w)
    assert int(ON.layer_acc(l, x.reshape(1, 30, 1, 1))[0, 0, 0, 0]) == int(x[0, c, y, xx])


def test_skip_add_in_int32_domain():
    rng = np.random.default_rng(5)
    l = dict(W.impala_resnet()[3])
    l["w"] = rng.integers(-127, 128, (l["out_c"], l["in_c"], 3, 3)).astype(np.int8)
    x = rng.integers(-128, 128, (2, l["in_c"], l["in_h"], l["in_w"])).astype(np.int8)
    skip = rng.integers(-128, 128, (2, l["out_c"], l["in_h"], l["in_w"])).astype(np.int8)
    r = rng.integers(0, 700, l["out_c"]).astype(np.int32)
    plain = ON.layer_acc(dict(l, skip_from=-1), x)
    both = ON.layer_acc(dict(l, skip_mul=r), x, skip)
    want = plain.astype(np.int64) + r.reshape(1, -1, 1, 1).astype(np.int64) * skip.astype(np.int64)
    assert np.array_equal(both.astype(np.int64), want)


# --------------------------------------------------------------------------
# fp64 de-quantised forward, layer by layer, with a different loop structure
# --------------------------------------------------------------------------

def _dequant_layer_fp64(l, x_q, skip_q=None, s_skip=None):
    """y = W_real * x_real + b (+ skip) in float64 via im2col + matmul."""
    b = x_q.shape[0]
    xr = x_q.astype(np.float64)
    if l["relu_in"]:
        xr = np.maximum(xr, 0)
    xr = xr * float(l["s_in"])
    wr = l["w"].astype(np.float64) * l["s_w"].astype(np.float64).reshape(-1, 1, 1, 1)
    if l["kind"] == "fc":
        y = xr.reshape(b, -1) @ wr.reshape(l["out_c"], -1).T
        y = y.reshape(b, -1, 1, 1)
    else:
        p = l["pad"]
        xp = np.pad(xr, ((0, 0), (0, 0), (p, p), (p, p)))
        win = np.lib.stride_tricks.sliding_window_view(xp, (l["kh"], l["kw"]), axis=(2, 3))
        win = win[:, :, ::l["stride"], ::l["stride"]]            # [b, c, oh, ow, kh, kw]
        cols = win.transpose(0, 2, 3, 1, 4, 5).reshape(b, win.shape[2], win.shape[3], -1)
        y = (cols @ wr.reshape(l["out_c"], -1).T).transpose(0, 3, 1, 2)
    y = y + l["bias"].astype(np.float64).reshape(1, -1, 1, 1)
    if skip_q is not None:
        eff = (l["skip_mul"].astype(np.float64) * float(l["s_in"]) * l["s_w"].astype(np.float64))
        y = y + skip_q.astype(np.float64) * eff.reshape(1, -1, 1, 1)
    if l["relu_out"]:
        y = np.maximum(y, 0)
    return y


def _check_against_dequant(pol, res, b):
    x = res["input_q"]
    for i, l in enumerate(pol["layers"]):
        if l["kind"] == "maxpool":
            x = res["activations"][i]
            continue
        xin = x.reshape(b, -1, 1, 1) if l["kind"] == "fc" else x
        skip = res["activations"][l["skip_from"]] if l["skip_from"] >= 0 else None
        y = _dequant_layer_fp64(l, xin, skip)
        if l["logits"]:
            mag = np.abs(y) + np.abs(l["bias"].astype(np.float64)).reshape(1, -1, 1, 1) + 1e-30
            assert np.all(np.abs(res["logits"].reshape(y.shape) - y) <= 1e-5 * (mag + 1.0))
        else:
            s = float(l["s_out"])
            q = res["activations"][i].astype(np.float64)
            err = np.abs(q * s - np.clip(y, -128 * s, 127 * s))
            assert err.max() <= (0.5 + 1e-3) * s, (i, err.max() / s)
            x = res["activations"][i]


@pytest.mark.parametrize("name,rows,batch", [("cartpole_mlp", 256, 32), ("lunarlander_mlp", 256, 16),
                                             ("student_cnn_b8192", 8, 3),
                                             ("impala_resnet_b16384", 6, 2)])
def test_each_layer_within_one_step_of_fp64_dequantised(name, rows, batch):
    c = W.config(name)
    pol = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                           W.calibration_batch(name, rows), c["prune24"])
    res = oracle.forward(pol, W.observations(name, batch), W.uniforms(name, batch))
    _check_against_dequant(pol, res, batch)


def test_tiny_odd_conv_net_against_fp64_dequantised():
    # odd sizes, stride 2 with padding, a max-pool and a residual connection
    rng = np.random.default_rng(11)
    mk = W._conv
    layers = [mk(3, 11, 9, 5, 3, 2, 1, relu_out=False), W._pool(5, 6, 5, 3, 2)]
    layers[0]["kw"] = 3
    layers += [mk(5, 2, 2, 5, 3, 1, 1, relu_in=True), mk(5, 2, 2, 5, 3, 1, 1, relu_out=False,
                                                          skip_from=1),
               W._fc(20, 7, relu_in=True), W._fc(7, 3, relu_out=False, logits=True)]
    params = []
    for l in layers:
        if l["kind"] == "maxpool":
            params.append(None)
            continue
        params.append(dict(w=rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])
                                                 ).astype(np.float32) * 0.3,
                           bias=rng.standard_normal(l["out_c"]).astype(np.float32) * 0.1))
    calib = rng.integers(0, 256, (16, 3, 11, 9), dtype=np.uint8)
    pol = oracle.calibrate("u8", (3, 11, 9), layers, params, calib)
    obs = rng.integers(0, 256, (5, 3, 11, 9), dtype=np.uint8)
    res = oracle.forward(pol, obs, rng.random(5, dtype=np.float32))
    _check_against_dequant(pol, res, 5)


# --------------------------------------------------------------------------
# structural special cases
# --------------------------------------------------------------------------

def test_conv_1x1_spatial_equals_fc_and_delta_kernel_shifts():
    rng = np.random.default_rng(2)
    x = rng.integers(-128, 128, (3, 6, 1, 1)).astype(np.int8)
    w = rng.integers(-127, 128, (4, 6, 1, 1)).astype(np.int8)
    conv = dict(kind="conv", in_c=6, in_h=1, in_w=1, out_c=4, kh=1, kw=1, stride=1, pad=0,
                relu_in=False, skip_from=-1, w=w)
    assert np.array_equal(ON.layer_acc(conv, x), ON.layer_acc(dict(conv, kind="fc"), x))
    # a kernel that is 1 at (ic=1, ky=2, kx=0) copies a shifted crop of channel 1
    x = rng.integers(-128, 128, (2, 2, 7, 6)).astype(np.int8)
    w = np.zeros((1, 2, 3, 3), np.int8)
    w[0, 1, 2, 0] = 1
    conv = dict(kind="conv", in_c=2, in_h=7, in_w=6, out_c=1, kh=3, kw=3, stride=1, pad=0,
                relu_in=False, skip_from=-1, w=w)
    assert np.array_equal(ON.layer_acc(conv, x)[:, 0], x[:, 1, 2:7, 0:4].astype(np.int32))
    # with padding 1 and stride 2 the same kernel reads x[2*oy+1, 2*ox-1], zero outside
    conv.update(pad=1, stride=2)
    got = ON.layer_acc(conv, x)[:, 0]
    want = np.zeros((2, 4, 3), np.int32)      # (7+2-3)//2+1 = 4, (6+2-3)//2+1 = 3
    for oy in range(4):
        for ox in range(3):
            iy, ix = 2 * oy + 1, 2 * ox - 1
            if 0 <= iy < 7 and 0 <= ix < 6:
                want[:, oy, ox] = x[:, 1, iy, ix]
    assert np.array_equal(got, want)


def test_zero_weights_give_requantised_bias_and_relu_precedes_clamp():
    l = dict(kind="fc", in_c=4, out_c=4, kh=1, kw=1, stride=1, pad=0, in_h=1, in_w=1,
             relu_in=False, relu_out=True, logits=False, skip_from=-1,
             w=np.zeros((4, 4, 1, 1), np.int8), s_w=np.ones(4, np.float32),
             bias=np.array([0.75, -0.75, 100.0, 0.25], np.float32), s_in=np.float32(1.0),
             s_out=np.float32(0.5))
    x = np.full((1, 4, 1, 1), 9, np.int8)
    y = ON.layer_float(l, ON.layer_acc(l, x))
    assert y.ravel().tolist() == [0.75, 0.0, 100.0, 0.25]
    assert ON.requant(y, l["s_out"]).ravel().tolist() == [2, 0, 127, 0]   # 1.5 -> 2, 0.5 -> 0
    y = ON.layer_float(dict(l, relu_out=False), ON.layer_acc(l, x))
    assert ON.requant(y, l["s_out"]).ravel().tolist() == [2, -2, 127, 0]  # -1.5 -> -2


def test_epilogue_uses_single_rounded_scale_product_and_fma():
    # k = fl(s_in * s_w) first, then one fused multiply-add: compare with exact arithmetic
    from fractions import Fraction as Fr
    s_in, s_w, bias = np.float32(0.0123), np.float32(0.00377), np.float32(-0.4321)
    acc = np.array([[[[33554433]], [[-7777777]], [[123]]]], np.int32).reshape(1, 3, 1, 1)
    l = dict(s_in=s_in, s_w=np.full(3, s_w, np.float32), bias=np.full(3, bias, np.float32),
             relu_out=False)
    y = ON.layer_float(l, acc).ravel()
    k = np.float32(s_in * s_w)
    for a, got in zip(acc.ravel(), y):
        exact = Fr(float(np.float32(a))) * Fr(float(k)) + Fr(float(bias))
        want = np.float32(float(exact))     # Fraction -> double is correctly rounded; double ->
        # float may double-round, so accept the neighbours only if the double was a tie
        assert got == want or abs(float(got) - float(exact)) <= abs(float(want) - float(exact))
    assert np.float32(33554433) == np.float32(33554432)  # the int -> float rounding is exercised


def test_maxpool_constant_and_window_rule():
    l = W._pool(2, 7, 7)
    x = np.full((1, 2, 7, 7), -5, np.int8)
    assert np.all(ON.maxpool(l, x) == -5) and ON.maxpool(l, x).shape == (1, 2, 3, 3)
    x[0, 1, 6, 6] = 100          # last row/col belongs to the last window (2*2+2 = 6)
    x[0, 0, 3, 3] = 50
    out = ON.maxpool(l, x)
    assert out[0, 1, 2, 2] == 100 and out[0, 1, 1, 1] == -5
    assert out[0, 0, 1, 1] == 50 and out[0, 0, 0, 0] == -5


def test_pool_and_requant_commute():
    # per channel (k > 0) acc -> q is monotone, so max then requant == requant then max
    rng = np.random.default_rng(13)
    acc = rng.integers(-40000, 40000, (4, 3, 9, 9)).astype(np.int32)
    l = dict(s_in=np.float32(0.013), s_w=np.array([0.002, 0.0007, 0.01], np.float32),
             bias=np.array([0.3, -0.2, 0.0], np.float32), relu_out=False)
    s_out = np.float32(0.031)
    q = ON.requant(ON.layer_float(l, acc), s_out)
    pool = W._pool(3, 9, 9)
    a = ON.maxpool(pool, q)
    win = np.lib.stride_tricks.sliding_window_view(acc, (3, 3), axis=(2, 3))[:, :, ::2, ::2]
    b = ON.requant(ON.layer_float(l, np.ascontiguousarray(win.max(axis=(-1, -2)))), s_out)
    assert np.array_equal(a, b)


# --------------------------------------------------------------------------
# sampler: brute force and invariants
# --------------------------------------------------------------------------

@pytest.mark.parametrize("a", [1, 2, 3, 18])
def test_sampler_against_library_softmax_and_searchsorted(a):
    from scipy.special import log_softmax
    rng = np.random.default_rng(a)
    z = (rng.standard_normal((40, a)) * 3).astype(np.float32)
    if a > 2:
        z[0, 1] = -200.0          # a zero-width bucket must never be chosen
        z[1, :] = 0.0             # uniform distribution
    lp = log_softmax(z.astype(np.float64), axis=1)
    cdf = np.cumsum(np.exp(lp), axis=1)
    grid = np.concatenate([np.linspace(0, 1, 41, endpoint=False), [0.99999994]]).astype(np.float32)
    for i in range(z.shape[0]):
        # the grid plus the fp32 neighbours of every bucket edge
        edges = cdf[i].astype(np.float32)
        us = np.concatenate([grid, edges, np.nextafter(edges, np.float32(0)),
                             np.nextafter(edges, np.float32(2))])
        us = us[(us >= 0) & (us < 1)].astype(np.float32)
        r = ON.sample(np.repeat(z[i:i + 1], len(us), 0), us)
        np.testing.assert_allclose(r["logp_all"], np.repeat(lp[i:i + 1], len(us), 0), atol=1e-12)
        want = np.minimum(np.searchsorted(cdf[i], us.astype(np.float64), side="right"), a - 1)
        near = np.min(np.abs(us.astype(np.float64)[:, None] - cdf[i][None, :]), axis=1) < 1e-12
        assert np.array_equal(r["actions"][~near], want[~near])
        np.testing.assert_allclose(r["margin"],
                                   np.min(np.abs(us.astype(np.float64)[:, None] - cdf[i][None]), 1),
                                   atol=1e-12)
        # invariants: a proper distribution; the action's bucket contains u; finite log-prob
        assert np.all(np.abs(np.exp(r["logp_all"]).sum(1) - 1) < 1e-9)
        assert np.all(np.isfinite(r["logp"])) and np.all(r["logp"] <= 0)
        assert np.all(r["logp"] == r["logp_all"][np.arange(len(us)), r["actions"]].astype(np.float32))
        if a > 2 and i == 0:
            assert not np.any(r["actions"] == 1)


# --------------------------------------------------------------------------
# quantiser, pruning, calibration
# --------------------------------------------------------------------------

def test_prune_2_4_brute_force_and_tie_break():
    rng = np.random.default_rng(17)
    w = rng.standard_normal((3, 8, 2, 2)).astype(np.float32)
    w[0, 0:4, 0, 0] = [1.0, -1.0, 1.0, 0.5]      # three-way tie: keep index 0 and 1
    p = oracle.prune_2_4(w)
    for oc in range(3):
        for ky in range(2):
            for kx in range(2):
                for g in range(2):
                    grp = w[oc, 4 * g:4 * g + 4, ky, kx]
                    keep = sorted(sorted(range(4), key=lambda j: (-abs(grp[j]), j))[:2])
                    for j in range(4):
                        want = grp[j] if j in keep else 0.0
                        assert p[oc, 4 * g + j, ky, kx] == want
    assert p[0, 0:4, 0, 0].tolist() == [1.0, -1.0, 0.0, 0.0]


def test_weight_quantiser_properties():
    rng = np.random.default_rng(19)
    w = rng.standard_normal((6, 5, 3, 3)).astype(np.float32)
    w[4] = 0
    q, s = oracle.quantise_weights(w)
    assert q.dtype == np.int8 and q.min() >= -127
    assert s[4] == 1.0 and np.all(q[4] == 0)
    for c in (0, 1, 2, 3, 5):
        assert np.abs(q[c]).max() == 127
        np.testing.assert_allclose(s[c] * 127, np.abs(w[c]).max(), rtol=1e-6)
        assert np.abs(q[c] * np.float64(s[c]) - w[c]).max() <= 0.5 * s[c] * (1 + 1e-5)


def test_calibration_scales_are_max_abs_over_127():
    name = "lunarlander_mlp"
    c = W.config(name)
    calib = W.calibration_batch(name, 128)
    pol = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name), calib)
    np.testing.assert_allclose(pol["s_input"] * 127, np.abs(calib).max(), rtol=1e-6)
    res = oracle.forward(pol, calib, np.zeros(128, np.float32))
    assert np.abs(res["input_q"]).max() == 127
    for i, l in enumerate(pol["layers"][:-1]):
        assert res["activations"][i].max() == 127        # the batch's own maximum maps to 127
        assert res["activations"][i].min() >= 0          # ReLU layers
        assert l["s_out"] == pol["layers"][i + 1]["s_in"]
    # a different batch may exceed the calibrated range and must saturate, not wrap
    big = (calib * 3).astype(np.float32)
    r2 = oracle.forward(pol, big, np.zeros(128, np.float32))
    assert r2["input_q"].max() == 127 and r2["input_q"].min() == -128


def test_resnet_policy_structure():
    name = "impala_resnet_b16384"
    c = W.config(name)
    pol = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                           W.calibration_batch(name, 4), True)
    assert pol["layers"][-2]["in_c"] == 2592
    for l in pol["layers"]:
        if l["w"] is None:
            assert l["s_out"] == l["s_in"]
            continue
        wk = l["w"].transpose(0, 2, 3, 1).reshape(l["out_c"], -1, 4)
        assert np.all((wk == 0).sum(-1) >= 2)             # 2:4 along K, c_in fastest
        if l["skip_from"] >= 0:
            r = l["skip_mul"]
            assert r.dtype == np.int32 and r.min() >= 1
            s_x = pol["layers"][l["skip_from"]]["s_out"]
            np.testing.assert_allclose(r * (l["s_in"] * l["s_w"]), s_x, rtol=0.02)


def test_batch_independence_and_permutation():
    name = "student_cnn_b8192"
    c = W.config(name)
    pol = oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                           W.calibration_batch(name, 4))
    obs, u = W.observations(name, 5), W.uniforms(name, 5)
    full = oracle.forward(pol, obs, u)
    perm = np.array([3, 0, 4, 2, 1])
    p = oracle.forward(pol, obs[perm], u[perm])
    assert np.array_equal(p["logits"], full["logits"][perm])
    assert np.array_equal(p["actions"], full["actions"][perm])
    one = oracle.forward(pol, obs[2:3], u[2:3])
    assert np.array_equal(one["logits"][0], full["logits"][2])
    for a, b in zip(one["activations"][:-1], full["activations"][:-1]):
        assert np.array_equal(a[0], b[2])
