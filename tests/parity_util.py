"""Shared helpers of the GPU parity tests: calibrated policies and the comparison itself."""
from __future__ import annotations

import functools

import numpy as np

import oracle
import workloads as W

# Tolerances of the parity bar: int8 activations and actions bit-exact (actions may differ only
# where the uniform lies within ACTION_MARGIN of a CDF edge; such cases are counted), log-probs
# (and entropies) within RTOL relative / ATOL absolute.  Logits and values are compared for
# EQUALITY: on both sides a logit is the single fp32 fma(float(acc), k, b) of the same integer
# accumulator and the same two fp32 constants, so there is exactly one correct bit pattern.
RTOL, ATOL, ACTION_MARGIN = 1e-5, 1e-6, 1e-5

# counters per label, summed over every compare() of the session; conftest prints them at the end
SESSION_STATS: dict = {}


@functools.lru_cache(maxsize=None)
def calibrated(name: str, rows: int = W.CALIBRATION_ROWS) -> dict:
    c = W.config(name)
    return oracle.calibrate(c["in_kind"], c["in_shape"], c["layers"], W.fp32_parameters(name),
                            W.calibration_batch(name, rows), c["prune24"])


def _tap_or_none(taps, layer, n):
    """A tap, or None where the (fused) plan never stores that tensor (status UNSUPPORTED)."""
    try:
        return taps(layer, n)
    except RuntimeError as e:
        if getattr(e, "status", None) == 2:
            return None
        raise


def compare(ref: dict, logits, actions, logp, taps=None, n_taps=None, label=None, value=None,
            entropy=None) -> dict:
    """Assert parity of one batch; returns counters.  ``taps(layer, n)`` reads int8 activations."""
    logits, actions, logp = (np.asarray(a) for a in (logits, actions, logp))
    b = logits.shape[0]
    stats = dict(states=b, int8_compared=0, int8_mismatch=0, taps_missing=0, logits_mismatch=0,
                 action_mismatch=0, action_mismatch_near_edge=0)
    if taps is not None:
        n = b if n_taps is None else n_taps
        got = _tap_or_none(taps, -1, n)
        if got is None:
            stats["taps_missing"] += 1
        else:
            want = ref["input_q"][:n].reshape(got.shape)
            stats["int8_compared"] += want.size
            stats["int8_mismatch"] += int((got != want).sum())
        for i, a in enumerate(ref["activations"]):
            if a is None:
                continue
            got = _tap_or_none(taps, i, n)
            if got is None:
                stats["taps_missing"] += 1
                continue
            want = a[:n].reshape(got.shape)
            bad = int((got != want).sum())
            stats["int8_compared"] += want.size
            stats["int8_mismatch"] += bad
            assert bad == 0, "layer %d: %d of %d int8 activations differ" % (i, bad, want.size)
        assert stats["int8_mismatch"] == 0
    stats["logits_mismatch"] = int((logits != ref["logits"]).sum())
    assert stats["logits_mismatch"] == 0, "%d of %d logits differ in their bits (max |diff| %.3g)" % (
        stats["logits_mismatch"], logits.size, np.abs(logits - ref["logits"]).max())
    if value is not None:
        assert np.array_equal(np.asarray(value), ref["value"]), "state values differ"
    if entropy is not None:
        np.testing.assert_allclose(np.asarray(entropy), ref["entropy"], rtol=RTOL, atol=ATOL)
    diff = actions != ref["actions"]
    stats["action_mismatch"] = int(diff.sum())
    stats["action_mismatch_near_edge"] = int((diff & (ref["margin"] < ACTION_MARGIN)).sum())
    assert stats["action_mismatch"] == stats["action_mismatch_near_edge"], \
        "%d actions differ away from a CDF edge" % (stats["action_mismatch"] -
                                                    stats["action_mismatch_near_edge"])
    same = ~diff
    np.testing.assert_allclose(logp[same], ref["logp"][same], rtol=RTOL, atol=ATOL)
    # where the action legitimately differs, the log-prob must be the one of the action taken
    for i in np.nonzero(diff)[0]:
        np.testing.assert_allclose(logp[i], ref["logp_all"][i, actions[i]], rtol=RTOL, atol=ATOL)
    assert np.all((actions >= 0) & (actions < logits.shape[1]))
    assert np.all(np.isfinite(logp)) and np.all(logp <= 0)
    if label is not None:
        tot = SESSION_STATS.setdefault(label, {k: 0 for k in stats})
        for k, v in stats.items():
            tot[k] += v
    return stats
