"""Seeded synthetic inputs for the int8 Actor policy-inference path.

This module only *draws inputs*: network shapes, fp32 parameters, observation
batches, per-state uniforms, and (for timing runs) ready-made int8 policies.
It contains none of the method's arithmetic (no quantisation rule, no
calibration, no forward pass), so that both the CPU oracle's tests and the
CUDA path's callers can use it without sharing anything else.

The shapes follow the paper's experimental section: the policy networks of
the table "network architecture and inference time" (input 4x84x84, conv
32(8)/64(4)/64(3) + fully connected, up to 18 actions) and the batch size of
160 states used in the introduction's time breakdown (Fig. 1).  Atari frames
and gym observations are replaced by iid draws of the same shape and dtype.
"""
from __future__ import annotations

import math
from typing import Dict, List

import numpy as np

# ---------------------------------------------------------------------------
# architectures
# ---------------------------------------------------------------------------


def _conv(in_c, in_h, in_w, out_c, k, stride, pad, relu_in=False, relu_out=True,
          skip_from=-1):
    return dict(kind="conv", in_c=in_c, in_h=in_h, in_w=in_w, out_c=out_c, kh=k, kw=k,
                stride=stride, pad=pad, relu_in=relu_in, relu_out=relu_out, logits=False,
                skip_from=skip_from)


def _fc(k, n, relu_in=False, relu_out=True, logits=False, value=False):
    return dict(kind="fc", in_c=k, in_h=1, in_w=1, out_c=n, kh=1, kw=1, stride=1, pad=0,
                relu_in=relu_in, relu_out=relu_out, logits=logits, skip_from=-1, value=value)


def with_value_head(layers: List[dict]) -> List[dict]:
    """The same architecture with a state-value output: the last layer gets one more output
    column (the value V(s)) after its action logits."""
    out = [dict(l) for l in layers]
    out[-1]["out_c"] += 1
    out[-1]["value"] = True
    return out


def _pool(c, h, w, k=3, stride=2):
    return dict(kind="maxpool", in_c=c, in_h=h, in_w=w, out_c=c, kh=k, kw=k, stride=stride,
                pad=0, relu_in=False, relu_out=False, logits=False, skip_from=-1)


def out_hw(layer) -> tuple:
    """Spatial size of a layer's output (floor division, as in every config here)."""
    if layer["kind"] == "fc":
        return 1, 1
    oh = (layer["in_h"] + 2 * layer["pad"] - layer["kh"]) // layer["stride"] + 1
    ow = (layer["in_w"] + 2 * layer["pad"] - layer["kw"]) // layer["stride"] + 1
    return oh, ow


def mlp(dims: List[int]) -> List[dict]:
    layers = []
    for i in range(len(dims) - 1):
        last = i == len(dims) - 2
        layers.append(_fc(dims[i], dims[i + 1], relu_out=not last, logits=last))
    return layers


def nature_cnn(c1=32, c2=64, c3=64, hidden=512, actions=18) -> List[dict]:
    """conv 8x8/4, conv 4x4/2, conv 3x3/1, fc, fc on 4x84x84 frames (no padding)."""
    return [
        _conv(4, 84, 84, c1, 8, 4, 0),
        _conv(c1, 20, 20, c2, 4, 2, 0),
        _conv(c2, 9, 9, c3, 3, 1, 0),
        _fc(c3 * 7 * 7, hidden),
        _fc(hidden, actions, relu_out=False, logits=True),
    ]


def impala_resnet(channels=(16, 32, 32), hidden=256, actions=18) -> List[dict]:
    """Three stacks of conv3x3(pad 1) + maxpool 3x3/2 + two residual blocks.

    A residual block on input x is ReLU -> conv -> ReLU -> conv, with x (before
    the ReLU) added to the second conv's int32 accumulators; ``skip_from`` names
    the layer whose int8 output is x.
    """
    layers: List[dict] = []
    c_in, h = 4, 84
    for c in channels:
        layers.append(_conv(c_in, h, h, c, 3, 1, 1, relu_out=False))
        layers.append(_pool(c, h, h))
        h = (h - 3) // 2 + 1
        for _ in range(2):
            x_idx = len(layers) - 1
            layers.append(_conv(c, h, h, c, 3, 1, 1, relu_in=True, relu_out=True))
            layers.append(_conv(c, h, h, c, 3, 1, 1, relu_out=False, skip_from=x_idx))
        c_in = c
    layers.append(_fc(c_in * h * h, hidden, relu_in=True))
    layers.append(_fc(hidden, actions, relu_out=False, logits=True))
    return layers


# name -> (input kind, input shape (C,H,W) or (D,1,1), layers, batch, obs distribution, id)
_FRAME = ("u8", (4, 84, 84))
CONFIGS: Dict[str, dict] = {
    "cartpole_mlp": dict(in_kind="f32", in_shape=(4, 1, 1), layers=mlp([4, 64, 64, 2]),
                         batch=160, obs="uniform", cfg_id=0, prune24=False),
    "lunarlander_mlp": dict(in_kind="f32", in_shape=(8, 1, 1), layers=mlp([8, 256, 256, 4]),
                            batch=4096, obs="normal", cfg_id=1, prune24=False),
    "nature_cnn_b160": dict(in_kind="u8", in_shape=(4, 84, 84), layers=nature_cnn(),
                            batch=160, obs="frames", cfg_id=2, prune24=False),
    "nature_cnn_b8192": dict(in_kind="u8", in_shape=(4, 84, 84), layers=nature_cnn(),
                             batch=8192, obs="frames", cfg_id=3, prune24=False),
    "student_cnn_b8192": dict(in_kind="u8", in_shape=(4, 84, 84),
                              layers=nature_cnn(16, 32, 32, 256), batch=8192, obs="frames",
                              cfg_id=33, prune24=False),
    "impala_resnet_b16384": dict(in_kind="u8", in_shape=(4, 84, 84), layers=impala_resnet(),
                                 batch=16384, obs="frames", cfg_id=4, prune24=True),
}

CALIBRATION_ROWS = 1024


def config(name: str) -> dict:
    return CONFIGS[name]


def n_actions(name: str) -> int:
    return CONFIGS[name]["layers"][-1]["out_c"]


def macs_per_state(name: str) -> int:
    total = 0
    for l in CONFIGS[name]["layers"]:
        if l["kind"] == "maxpool":
            continue
        oh, ow = out_hw(l)
        total += oh * ow * l["out_c"] * l["in_c"] * l["kh"] * l["kw"]
    return total


def input_bytes_per_state(name: str) -> int:
    c = CONFIGS[name]
    n = int(np.prod(c["in_shape"]))
    return n if c["in_kind"] == "u8" else 4 * n


# ---------------------------------------------------------------------------
# seeded draws
# ---------------------------------------------------------------------------


def fp32_parameters(name: str, seed: int | None = None) -> List[dict | None]:
    """Kaiming-normal fp32 weights (std = sqrt(2 / fan_in)), bias ~ N(0, std 0.01).

    One entry per layer (None for max-pool), weights in OIHW order.
    """
    c = CONFIGS[name]
    rng = np.random.default_rng(1000 + c["cfg_id"] if seed is None else seed)
    out: List[dict | None] = []
    for l in c["layers"]:
        if l["kind"] == "maxpool":
            out.append(None)
            continue
        fan_in = l["in_c"] * l["kh"] * l["kw"]
        w = rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])) * math.sqrt(2.0 / fan_in)
        b = rng.standard_normal(l["out_c"]) * 0.01
        out.append(dict(w=w.astype(np.float32), bias=b.astype(np.float32)))
    return out


def parameters_for(layers: List[dict], seed: int) -> List[dict | None]:
    """The draw of ``fp32_parameters`` for any list of layer shapes."""
    rng = np.random.default_rng(seed)
    out: List[dict | None] = []
    for l in layers:
        if l["kind"] == "maxpool":
            out.append(None)
            continue
        fan_in = l["in_c"] * l["kh"] * l["kw"]
        w = rng.standard_normal((l["out_c"], l["in_c"], l["kh"], l["kw"])) * math.sqrt(2.0 / fan_in)
        b = rng.standard_normal(l["out_c"]) * 0.01
        out.append(dict(w=w.astype(np.float32), bias=b.astype(np.float32)))
    return out


def rollouts(n_steps: int, batch: int, seed: int, actions: int = 18, p_done: float = 0.05,
             gamma: float = 0.99) -> dict:
    """Synthetic Actor rollouts for the Corrector, time-major float32 [n_steps, batch]:
    behaviour and target log-probs of the actions taken (log of a Dirichlet-like draw, so the
    importance ratios fall on both sides of 1), rewards in {-1, 0, 1} as clipped Atari rewards
    are, value estimates ~ N(0, 1), a bootstrap value per rollout and per-step discounts
    (gamma, or 0 where an episode ends)."""
    rng = np.random.default_rng(seed)
    shape = (n_steps, batch)
    lo = np.log(rng.dirichlet(np.ones(actions), size=shape)[..., 0] + 1e-6)
    ls = np.log(rng.dirichlet(np.ones(actions), size=shape)[..., 0] + 1e-6)
    return dict(logp_smaller=ls.astype(np.float32), logp_original=lo.astype(np.float32),
                rewards=rng.integers(-1, 2, size=shape).astype(np.float32),
                values=rng.standard_normal(shape).astype(np.float32),
                bootstrap=rng.standard_normal(batch).astype(np.float32),
                discounts=np.where(rng.random(shape) < p_done, 0.0, gamma).astype(np.float32),
                gamma=gamma)


def observations(name: str, batch: int | None = None, seed: int | None = None) -> np.ndarray:
    """A batch of states: uint8 frames [B,4,84,84] or fp32 vectors [B,D]."""
    c = CONFIGS[name]
    b = c["batch"] if batch is None else batch
    rng = np.random.default_rng(3000 + c["cfg_id"] if seed is None else seed)
    if c["obs"] == "frames":
        return rng.integers(0, 256, size=(b,) + tuple(c["in_shape"]), dtype=np.uint8)
    d = c["in_shape"][0]
    if c["obs"] == "uniform":
        return rng.uniform(-1.0, 1.0, size=(b, d)).astype(np.float32)
    return rng.standard_normal((b, d)).astype(np.float32)


def calibration_batch(name: str, rows: int = CALIBRATION_ROWS) -> np.ndarray:
    return observations(name, rows, seed=2000 + CONFIGS[name]["cfg_id"])


def uniforms(name: str, batch: int | None = None, seed: int | None = None) -> np.ndarray:
    """One U[0,1) fp32 number per state for inverse-CDF sampling."""
    c = CONFIGS[name]
    b = c["batch"] if batch is None else batch
    rng = np.random.default_rng(4000 + c["cfg_id"] if seed is None else seed)
    return rng.random(b, dtype=np.float32)


def drawn_int8_policy(name: str, seed: int | None = None) -> dict:
    """An int8 policy drawn directly, for timing runs that have no calibrator at hand.

    Weights are iid rounded normals clipped to [-127, 127]; per-channel weight
    scales, biases, activation scales and residual multipliers are drawn or set
    to the magnitudes a Kaiming-initialised ReLU network has (second moment of
    the activations is preserved from layer to layer).  The result has the same
    structure as a calibrated policy: a dict with ``in_kind``, ``in_shape``,
    ``s_input`` and ``layers`` (each with ``w`` int8 OIHW, ``s_w``, ``bias``,
    ``s_in``, ``s_out``, ``skip_mul``).  With ``prune24`` configs, two of every
    four consecutive K positions (c_in fastest within a tap) are zero.
    """
    c = CONFIGS[name]
    rng = np.random.default_rng(5000 + c["cfg_id"] if seed is None else seed)
    m2 = 1.0 if c["obs"] == "normal" else 1.0 / 3.0
    s_input = np.float32(4.0 / 127.0) if c["obs"] == "normal" else np.float32(1.0 / 127.0)
    layers = []
    scales: List[np.float32] = []
    s_prev = s_input
    for i, l in enumerate(c["layers"]):
        e = dict(l)
        if l["kind"] == "maxpool":
            e.update(w=None, s_w=None, bias=None, s_in=s_prev, s_out=s_prev, skip_mul=None)
            layers.append(e)
            scales.append(s_prev)
            continue
        oc, ic, kh, kw = l["out_c"], l["in_c"], l["kh"], l["kw"]
        fan_in = ic * kh * kw
        w = np.clip(np.rint(rng.standard_normal((oc, ic, kh, kw)) * (127.0 / 4.0)), -127, 127)
        if c["prune24"]:
            # K order (kh, kw, c_in), c_in fastest: zero two random positions of each 4
            wk = w.transpose(0, 2, 3, 1).reshape(oc, -1, 4)
            order = np.argsort(rng.random(wk.shape), axis=-1)
            np.put_along_axis(wk, order[..., :2], 0.0, axis=-1)
            w = wk.reshape(oc, kh, kw, ic).transpose(0, 3, 1, 2)
        e["w"] = np.ascontiguousarray(w).astype(np.int8)
        e["s_w"] = np.full(oc, 4.0 * math.sqrt(2.0 / fan_in) / 127.0, np.float32) * \
            rng.uniform(0.8, 1.2, oc).astype(np.float32)
        e["bias"] = (rng.standard_normal(oc) * 0.01).astype(np.float32)
        e["s_in"] = s_prev
        grow = 2.0 if l["skip_from"] >= 0 else 1.0
        m2 *= grow
        e["s_out"] = np.float32(1.0) if l["logits"] else np.float32(5.0 * math.sqrt(2.0 * m2) / 127.0)
        e["skip_mul"] = None
        if l["skip_from"] >= 0:
            e["skip_mul"] = rng.integers(60, 200, oc).astype(np.int32)
        layers.append(e)
        scales.append(e["s_out"])
        s_prev = e["s_out"]
    return dict(in_kind=c["in_kind"], in_shape=tuple(c["in_shape"]), s_input=s_input, layers=layers)
