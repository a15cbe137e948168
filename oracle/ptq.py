"""Post-training quantisation and calibration (TEST INFRASTRUCTURE).

The paper's Compressor applies post-training quantisation to the policy the
Actors run (Section 2.2, paragraph "Parameter Quantization") and, for one
workload here, prunes weights first (paragraph "Structured Pruning" motivates
pruning; the 2-of-4 pattern is the workload's).  The scheme is the plain one:
symmetric int8, one scale per output channel for weights (max|w| / 127), one
scale per tensor for activations, calibrated as the max-abs of the epilogue
float over a seeded batch that is pushed through the already-quantised
preceding layers.
"""
from __future__ import annotations

import numpy as np

from . import net as F


def prune_2_4(w: np.ndarray) -> np.ndarray:
    """Keep the 2 largest-|w| of every 4 consecutive K positions, zero the rest.

    K runs over (kh, kw, c_in) with c_in fastest (for an fc layer: the input
    index).  Ties keep the lower index.  ``w`` is fp32 OIHW; returns a copy.
    """
    oc, ic, kh, kw = w.shape
    wk = np.ascontiguousarray(w.transpose(0, 2, 3, 1)).reshape(oc, -1)
    assert wk.shape[1] % 4 == 0
    g = wk.reshape(oc, -1, 4).copy()
    # stable sort on -|w| keeps the lower index first among equals
    order = np.argsort(-np.abs(g), axis=-1, kind="stable")
    np.put_along_axis(g, order[..., 2:], np.float32(0), axis=-1)
    return np.ascontiguousarray(g.reshape(oc, kh, kw, ic).transpose(0, 3, 1, 2))


def quantise_weights(w: np.ndarray) -> tuple:
    """s_w[c] = max|w[c]| / 127 (1.0 for an all-zero channel); q = clip(rint(w / s_w), +-127)."""
    w = w.astype(np.float32)
    oc = w.shape[0]
    mx = np.abs(w.reshape(oc, -1)).max(axis=1).astype(np.float32)
    s_w = np.where(mx > 0, mx / np.float32(127.0), np.float32(1.0)).astype(np.float32)
    q = np.rint(w / s_w.reshape(oc, 1, 1, 1).astype(np.float32))
    return np.clip(q, -127, 127).astype(np.int8), s_w


def _scale_of(maxabs) -> np.float32:
    m = np.float32(maxabs)
    return np.float32(m / np.float32(127.0)) if m > 0 else np.float32(1.0)


def calibrate(in_kind: str, in_shape, layers, params, calib_obs: np.ndarray,
              prune24: bool = False) -> dict:
    """Quantise fp32 parameters and calibrate every activation scale.

    ``layers`` are architecture dicts (kind, shapes, relu flags, skip_from),
    ``params`` the matching fp32 {w, bias} (None for max-pool).  Returns the
    policy dict the forward pass and the device library consume.
    """
    b = calib_obs.shape[0]
    if in_kind == "u8":
        x_real = calib_obs.astype(np.float32) / np.float32(255.0)
    else:
        x_real = calib_obs.astype(np.float32)
    s_input = _scale_of(np.abs(x_real).max())
    x = F.ingest(in_kind, calib_obs, s_input).reshape((b,) + tuple(in_shape))
    out_layers, outs, scales = [], [], []
    s_prev = s_input
    for l, p in zip(layers, params):
        e = dict(l)
        if l["kind"] == "maxpool":
            e.update(w=None, s_w=None, bias=None, skip_mul=None, s_in=s_prev, s_out=s_prev)
            x = F.maxpool(e, x)
        else:
            w = p["w"].astype(np.float32)
            if prune24:
                w = prune_2_4(w)
            e["w"], e["s_w"] = quantise_weights(w)
            e["bias"] = p["bias"].astype(np.float32)
            e["s_in"] = s_prev
            e["skip_mul"] = None
            skip = None
            if l["skip_from"] >= 0:
                # integer multiplier that brings the skip tensor (scale s_x) onto the
                # accumulator's grid (s_in * s_w[c]): r = rint(s_x / (s_in * s_w[c]))
                s_x = np.float32(scales[l["skip_from"]])
                k = (np.float32(s_prev) * e["s_w"]).astype(np.float32)
                e["skip_mul"] = np.clip(np.rint(s_x / k), 0, 32767).astype(np.int32)
                skip = outs[l["skip_from"]]
            if l["kind"] == "fc":
                x = x.reshape(b, -1, 1, 1)
            e["s_out"] = np.float32(1.0)
            acc = F.layer_acc(e, x, skip)
            y = F.layer_float(e, acc)
            if not l["logits"]:
                e["s_out"] = _scale_of(np.abs(y).max())
                x = F.requant(y, e["s_out"])
        out_layers.append(e)
        outs.append(x)
        scales.append(e["s_out"])
        s_prev = e["s_out"]
    return dict(in_kind=in_kind, in_shape=tuple(in_shape), s_input=s_input, layers=out_layers)
