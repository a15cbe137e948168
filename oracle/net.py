"""Whole forward pass of a quantised policy, layer by layer (TEST INFRASTRUCTURE).

Composes the naive C routines in the order the path runs them: input
quantisation, then per layer contraction -> optional int32 residual add ->
float epilogue -> requantise (or stop at the float logits), then sampling.
Activations are int8 NCHW numpy arrays; a policy is a dict with ``in_kind``,
``in_shape``, ``s_input`` and ``layers`` (see ``oracle.ptq.calibrate``).
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .clib import lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def ingest(in_kind: str, obs: np.ndarray, s_input) -> np.ndarray:
    """Quantise observations to int8 with the per-tensor input scale."""
    obs = np.ascontiguousarray(obs)
    q = np.empty(obs.shape, np.int8)
    if in_kind == "u8":
        assert obs.dtype == np.uint8
        lib().oracle_ingest_u8(_p(obs), C.c_int64(obs.size), C.c_float(s_input), _p(q))
    else:
        assert obs.dtype == np.float32
        lib().oracle_ingest_f32(_p(obs), C.c_int64(obs.size), C.c_float(s_input), _p(q))
    return q


def out_hw(l) -> tuple:
    if l["kind"] == "fc":
        return 1, 1
    return ((l["in_h"] + 2 * l["pad"] - l["kh"]) // l["stride"] + 1,
            (l["in_w"] + 2 * l["pad"] - l["kw"]) // l["stride"] + 1)


def layer_acc(l, x: np.ndarray, skip: np.ndarray | None = None) -> np.ndarray:
    """int32 accumulators of a conv / fc layer, residual add included."""
    b = x.shape[0]
    x = np.ascontiguousarray(x, np.int8)
    w = np.ascontiguousarray(l["w"], np.int8)
    oh, ow = out_hw(l)
    acc = np.empty((b, l["out_c"], oh, ow), np.int32)
    if l["kind"] == "conv":
        assert x.shape[1:] == (l["in_c"], l["in_h"], l["in_w"]), (x.shape, l)
        lib().oracle_conv_acc(_p(x), b, l["in_c"], l["in_h"], l["in_w"], _p(w), l["out_c"],
                              l["kh"], l["kw"], l["stride"], l["pad"], int(l["relu_in"]), _p(acc))
    else:
        assert x.size == b * l["in_c"], (x.shape, l["in_c"])
        lib().oracle_fc_acc(_p(x), b, l["in_c"], _p(w), l["out_c"], int(l["relu_in"]), _p(acc))
    if l["skip_from"] >= 0:
        skip = np.ascontiguousarray(skip, np.int8)
        assert skip.shape == acc.shape
        r = np.ascontiguousarray(l["skip_mul"], np.int32)
        lib().oracle_skip_add(_p(acc), _p(skip), _p(r), b, l["out_c"], oh * ow)
    return acc


def layer_float(l, acc: np.ndarray) -> np.ndarray:
    """Epilogue float y (ReLU applied if the layer has it); the logits of a final layer."""
    b, c = acc.shape[:2]
    y = np.empty(acc.shape, np.float32)
    s_w = np.ascontiguousarray(l["s_w"], np.float32)
    bias = np.ascontiguousarray(l["bias"], np.float32)
    lib().oracle_epilogue_float(_p(acc), b, c, acc.shape[2] * acc.shape[3], C.c_float(l["s_in"]),
                                _p(s_w), _p(bias), int(l["relu_out"]), _p(y))
    return y


def requant(y: np.ndarray, s_out) -> np.ndarray:
    q = np.empty(y.shape, np.int8)
    lib().oracle_requant(_p(np.ascontiguousarray(y)), C.c_int64(y.size), C.c_float(s_out), _p(q))
    return q


def maxpool(l, x: np.ndarray) -> np.ndarray:
    b = x.shape[0]
    oh, ow = out_hw(l)
    out = np.empty((b, l["in_c"], oh, ow), np.int8)
    lib().oracle_maxpool(_p(np.ascontiguousarray(x, np.int8)), b, l["in_c"], l["in_h"], l["in_w"],
                         l["kh"], l["stride"], _p(out))
    return out


def sample(logits: np.ndarray, u: np.ndarray) -> dict:
    logits = np.ascontiguousarray(logits, np.float32)
    u = np.ascontiguousarray(u, np.float32)
    b, a = logits.shape
    logp_all = np.empty((b, a), np.float64)
    actions = np.empty(b, np.int32)
    logp = np.empty(b, np.float32)
    margin = np.empty(b, np.float64)
    lib().oracle_sample(_p(logits), b, a, _p(u), _p(logp_all), _p(actions), _p(logp), _p(margin))
    return dict(logp_all=logp_all, actions=actions, logp=logp, margin=margin)


def entropy(logits: np.ndarray) -> np.ndarray:
    """Per-state entropy of softmax(logits), float64."""
    logits = np.ascontiguousarray(logits, np.float32)
    b, a = logits.shape
    h = np.empty(b, np.float64)
    lib().oracle_entropy(_p(logits), b, a, _p(h))
    return h


def kl(logits_original: np.ndarray, logits_smaller: np.ndarray) -> np.ndarray:
    """Per-state KL(pi_original || pi_smaller) from two logit matrices, float64."""
    lo = np.ascontiguousarray(logits_original, np.float32)
    ls = np.ascontiguousarray(logits_smaller, np.float32)
    assert lo.shape == ls.shape
    b, a = lo.shape
    out = np.empty(b, np.float64)
    lib().oracle_kl(_p(lo), _p(ls), b, a, _p(out))
    return out


def forward(policy: dict, obs: np.ndarray, u: np.ndarray, keep: bool = True) -> dict:
    """Forward + sampling.  Returns logits, actions, logp, logp_all, margin, entropy and, with
    ``keep``, ``input_q`` and ``activations`` (one int8 NCHW array per non-final layer).

    A final layer with ``value`` set has one output column more than there are actions: that
    last column is the state value V(s) (the same single fma as a logit, no requantisation);
    it is returned as ``value`` and takes no part in the softmax."""
    b = obs.shape[0]
    x = ingest(policy["in_kind"], obs, policy["s_input"]).reshape((b,) + tuple(policy["in_shape"]))
    outs = []
    input_q = x
    logits = value = None
    for l in policy["layers"]:
        if l["kind"] == "maxpool":
            x = maxpool(l, x)
        else:
            if l["kind"] == "fc":
                x = x.reshape(b, -1, 1, 1)
            acc = layer_acc(l, x, outs[l["skip_from"]] if l["skip_from"] >= 0 else None)
            y = layer_float(l, acc)
            if l["logits"]:
                logits = y.reshape(b, -1)
                if l.get("value"):
                    value = np.ascontiguousarray(logits[:, -1])
                    logits = np.ascontiguousarray(logits[:, :-1])
                outs.append(None)
                break
            x = requant(y, l["s_out"])
        outs.append(x)
    res = sample(logits, u)
    res["logits"] = logits
    res["entropy"] = entropy(logits)
    if value is not None:
        res["value"] = value
    if keep:
        res["input_q"] = input_q
        res["activations"] = outs
    return res


def forward_mixed(smaller: dict, original: dict, obs: np.ndarray, u: np.ndarray,
                  u_select: np.ndarray, alpha: float) -> dict:
    """Per-state choice between two policies: state i runs ``smaller`` when
    ``u_select[i] < alpha`` and ``original`` otherwise (the Actor uses the small network with
    probability alpha).  Returns the chosen network's outputs per state plus ``use_smaller``."""
    rs = forward(smaller, obs, u, keep=False)
    ro = forward(original, obs, u, keep=False)
    pick = np.asarray(u_select, np.float32) < np.float32(alpha)
    out = dict(use_smaller=pick)
    for k in ("logits", "actions", "logp", "logp_all", "margin", "entropy", "value"):
        if k in rs and k in ro:
            sel = pick.reshape((-1,) + (1,) * (rs[k].ndim - 1))
            out[k] = np.where(sel, rs[k], ro[k])
    return out
